import json
import sys
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import load_oracle
    return load_oracle("parity")


@pytest.fixture(scope="session")
def golden():
    with open(ROOT / "tests" / "golden" / "hand_cases.json") as f:
        return json.load(f)


def f32_to_bf16_bits(x) -> np.ndarray:
    """Test-side helper: exact conversion of values already representable in bf16."""
    u = np.asarray(x, np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "value not representable in bf16"
    return (u >> 16).astype(np.uint16)


def torch_bf16_to_bits(t) -> np.ndarray:
    import torch
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
