"""bitlinear_forward_static: the forward for callers that may not allocate device memory.

Such a caller (a plug-in inside another framework's memory pool, a loop that must stay off the allocator)
hands over inputs and an output buffer only; the scratch is part of the library.  The checks: two calls
in a row through the C ABI give exactly what bitlinear_forward gives with a caller workspace, shapes that
do not fit the built-in scratch are refused before anything is launched, and the call really allocates
nothing.  This file sorts last on purpose, so that a run that stops at the first failure has already
been through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu

REL_TOL, ABS_TOL = 1e-2, 1e-3


def _as_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,K,N", [(5, 3200, 1024), (1, 4096, 4096), (130, 1536, 512)])
def test_static_forward_matches_forward_twice_in_a_row(M, K, N):
    from paper_2402_17764_b200 import build
    build.build()
    L = B.load_library()
    W = S.latent_weights(N, K, 11).cuda()
    packed, gamma = B.quantize_weights(W)
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):  # the second call finds the scratch as the first one left it
        X = S.activations(M, K, 100 + call, outlier_frac=0.01, outlier_scale=20.0).cuda()
        want = B.forward(packed, gamma, X, N)
        got = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        st = L.bitlinear_forward_static(packed.data_ptr(), gamma.data_ptr(), X.data_ptr(), M, K, N, got.data_ptr(), stream)
        assert st == B.OK
        assert torch.cuda.memory_allocated() == before, "the call must not allocate through torch"
        torch.cuda.synchronize()
        a, b = _as_f64(got), _as_f64(want)
        assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b)), f"call {call}: outside 1e-2 rel / 1e-3 abs"
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"call {call}: expected identical bf16 bits"


def test_static_forward_refuses_what_does_not_fit():
    L = B.load_library()
    limit = 8 << 20
    M, K, N = 64, 4096, 65536  # the int32 scratch alone is 16 MiB
    assert B.workspace_bytes(M, N, K) > limit
    fake = 0x1000  # never dereferenced: the size check comes first
    assert L.bitlinear_forward_static(fake, fake, fake, M, K, N, fake, None) == B.ERR_WORKSPACE
    assert L.bitlinear_forward_static(fake, fake, fake, 1, 24, 16, fake, None) == B.ERR_SHAPE
