"""CPU-only checks of the boundary: the library builds, loads, exports every declared symbol,
validates arguments on the host, and refuses to run without an sm_100 device."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2402_17764_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_functions():
    text = (ROOT / "include" / "bitlinear.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bitlinear_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 13
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/bitlinear.h but not exported"
    from paper_2402_17764_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_host_only_functions(lib):
    from paper_2402_17764_b200 import binding as B
    assert B.status_string(0) == "ok"
    assert "timed out" in B.status_string(B.ERR_TIMEOUT)
    assert B.status_string(12345) == "unknown status"
    # packed size: N and K padded to 64, two bits per weight
    assert B.packed_bytes(4096, 1536) == 4096 * 1536 // 4 == 1572864
    assert B.packed_bytes(3200, 8640) == 3200 * 8640 // 4
    assert B.packed_bytes(1040, 144) == 1088 * 192 // 4
    assert B.packed_bytes(16, 16) == 64 * 64 // 4
    assert B.packed_bytes(17, 128) == 0 and B.packed_bytes(16, 24) == 0 and B.packed_bytes(16, 131072 + 16) == 0
    assert B.workspace_bytes(8, 4096, 1536) >= 8 * 1536 + 8 * 8 + 256
    assert B.workspace_bytes(8, 4096, 1536) % 256 == 0
    assert B.workspace_bytes(-1, 4096, 1536) == 0


def test_argument_errors_are_reported_before_any_device_work(lib):
    from paper_2402_17764_b200 import binding as B
    L = lib
    null = None
    fake = 0x1000  # non-null, 16-byte aligned; never dereferenced because validation or the arch check fails first
    assert L.bitlinear_quantize_weights(null, 16, 16, 1e-5, fake, fake, null) == B.ERR_ARG
    assert L.bitlinear_quantize_weights(fake, 15, 16, 1e-5, fake, fake, null) == B.ERR_SHAPE
    assert L.bitlinear_quantize_weights(fake, 16, 24, 1e-5, fake, fake, null) == B.ERR_SHAPE
    assert L.bitlinear_quantize_weights(fake + 4, 16, 16, 1e-5, fake, fake, null) == B.ERR_ALIGN
    assert L.bitlinear_quantize_weights(fake, 16, 16, -1.0, fake, fake, null) == B.ERR_ARG
    assert L.bitlinear_quantize_acts(fake, 1, 16, null, fake, fake, null) == B.ERR_ARG
    assert L.bitlinear_quantize_acts(null, -1, 16, null, null, null, null) == B.ERR_SHAPE
    assert L.bitlinear_quantize_acts(fake, 1 << 21, 16, fake, fake, fake, null) == B.ERR_SHAPE
    assert L.bitlinear_forward(fake, fake, fake, 1, 16, 16, fake, fake + 16, 1 << 20, null) == B.ERR_ALIGN
    assert L.bitlinear_forward(fake, fake, fake, 1, 16, 16, fake, fake, 16, null) == B.ERR_WORKSPACE
    assert L.bitlinear_matmul_i32(fake, fake, 9, 16, 16, fake, B.PATH_DP4A, fake, 1 << 20, null) == B.ERR_SHAPE
    assert L.bitlinear_matmul_i32(fake, fake, 65, 16, 16, fake, B.PATH_MMA, fake, 1 << 20, null) == B.ERR_SHAPE
    assert L.bitlinear_matmul_i32(fake, fake, 1, 16, 16, fake, 7, fake, 1 << 20, null) == B.ERR_ARG
    assert L.bitlinear_poll_status(null, null, None) == B.ERR_ARG
    assert L.bitlinear_forward_sequence(null, null) == B.ERR_ARG
    L.bitlinear_sequence_destroy(null)  # allowed
    descs = (B.LayerDesc * 1)(B.LayerDesc(fake, fake, fake, fake, 65, 16, 16))
    assert L.bitlinear_sequence_workspace_bytes(descs, 1) > 0  # any M from 1 to 2^20 is a sequence entry
    for bad_m in (0, (1 << 20) + 1):
        descs = (B.LayerDesc * 1)(B.LayerDesc(fake, fake, fake, fake, bad_m, 16, 16))
        assert L.bitlinear_sequence_workspace_bytes(descs, 1) == 0


def test_no_cpu_fallback():
    """Valid arguments on a machine without an sm_100 GPU must fail loudly, not compute on the host."""
    import torch
    if torch.cuda.is_available() and torch.cuda.get_device_capability()[0] == 10:
        pytest.skip("an sm_100 device is present")
    from paper_2402_17764_b200 import binding as B
    L = B.load_library()
    fake = 0x1000
    assert L.bitlinear_quantize_weights(fake, 16, 16, 1e-5, fake, fake, None) == B.ERR_ARCH
    assert L.bitlinear_forward(fake, fake, fake, 1, 16, 16, fake, fake, 1 << 20, None) == B.ERR_ARCH


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    from paper_2402_17764_b200 import binding as B
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(FileNotFoundError):
        B.load_library()


def test_product_path_does_not_import_the_oracle():
    pkg = ROOT / "paper_2402_17764_b200"
    for f in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu")) + list(pkg.rglob("*.cuh")):
        text = f.read_text()
        assert not re.search(r"(^|\n)\s*(import|from)\s+oracle|oracle[/.]|liboracle|libbitlinear_oracle", text), \
            f"{f} reaches into the oracle"
