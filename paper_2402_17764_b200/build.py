"""Builds the CUDA library in-tree with nvcc for sm_100a.  Usage: python -m paper_2402_17764_b200.build"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libbitlinear_b200.so"
SOURCES = ["bitlinear_api.cu", "pack_weights.cu", "quantize_acts.cu", "decode_gemv.cu", "prefill_gemm.cu", "decode_tc.cu", "peak_probe.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "bitlinear.h"]
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every kernel for sm_100a into one shared library next to this file."""
    if not force and not needs_build():
        return LIB
    objs = []
    obj_dir = PKG / "_build"
    obj_dir.mkdir(exist_ok=True)
    common = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-Xcompiler", "-fPIC", "--cudart", "static",
    ]
    if verbose:
        common += ["-Xptxas", "-v"]
    procs = []
    for src in SOURCES:
        obj = obj_dir / (src + ".o")
        objs.append(str(obj))
        procs.append(subprocess.Popen(common + ["-c", str(CSRC / src), "-o", str(obj)]))
    failed = [p.args for p in procs if p.wait() != 0]
    if failed:
        raise RuntimeError(f"nvcc failed: {failed[0]}")
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.run([_nvcc(), "-shared", "--cudart", "static", "-o", str(tmp), *objs], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
