"""bitlinear_forward_static: the forward for callers that may not allocate device memory.

Such a caller (a plug-in inside another framework's memory pool, a loop that must stay off the allocator)
hands over inputs and an output buffer only; the scratch is part of the library.  The checks: two calls
in a row through the C ABI give exactly what bitlinear_forward gives with a caller workspace and what the CPU
oracle gives, also when the scratch still holds another, larger shape's leftovers and the new shape has ragged
tiles; shapes that do not fit the built-in scratch are refused before anything is launched, and the call really
allocates nothing.  This file sorts last on purpose, so that a run that stops at the first failure has already
been through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from conftest import torch_bf16_to_bits
from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu

REL_TOL, ABS_TOL = 1e-2, 1e-3


def _as_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _oracle():
    from oracle import load_oracle
    return load_oracle("timing")


@pytest.mark.parametrize("M,K,N", [(5, 3200, 1024), (1, 4096, 4096), (130, 1536, 512), (7, 144, 48)])
def test_static_forward_matches_forward_twice_in_a_row(M, K, N):
    from paper_2402_17764_b200 import build
    build.build()
    L = B.load_library()
    W = S.latent_weights(N, K, 11)
    T_ref, g_ref = _oracle().quantize_weights(W.numpy())
    packed, gamma = B.quantize_weights(W.cuda())
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):  # the second call finds the scratch as the first one left it
        X = S.activations(M, K, 100 + call, outlier_frac=0.01, outlier_scale=20.0)
        want_oracle = _oracle().forward(T_ref, g_ref, torch_bf16_to_bits(X))
        X = X.cuda()
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
        assert np.array_equal(torch_bf16_to_bits(got), want_oracle), f"call {call}: bf16 bits differ from the oracle"


def test_static_forward_after_a_larger_shape_left_its_scratch():
    """The scratch is shared by all calls.  A large streaming shape fills it with partial sums, lists and activations;
    a ragged GEMM shape (31 tokens, K and N no multiples of 64) and a ragged streaming shape that follow at once must
    still give the oracle's bits."""
    L = B.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    orc = _oracle()

    def run(M, K, N, seed):
        W = S.latent_weights(N, K, seed)
        X = S.activations(M, K, seed, outlier_frac=0.01, outlier_scale=20.0)
        T_ref, g_ref = orc.quantize_weights(W.numpy())
        want = orc.forward(T_ref, g_ref, torch_bf16_to_bits(X))
        packed, gamma = B.quantize_weights(W.cuda())
        got = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
        Xd = X.cuda()
        st = L.bitlinear_forward_static(packed.data_ptr(), gamma.data_ptr(), Xd.data_ptr(), M, K, N, got.data_ptr(), stream)
        assert st == B.OK
        torch.cuda.synchronize()
        assert np.array_equal(torch_bf16_to_bits(got), want), f"({M},{K},{N}): bf16 bits differ from the oracle"

    for big, small in (((16, 8640, 3200), (31, 144, 4112)), ((8, 8640, 3200), (7, 144, 48)), ((64, 1536, 4096), (3, 80, 528))):
        run(*big, seed=21)
        run(*small, seed=22)


def test_static_forward_refuses_what_does_not_fit():
    L = B.load_library()
    limit = 8 << 20
    M, K, N = 64, 4096, 65536  # the int32 scratch alone is 16 MiB
    assert B.workspace_bytes(M, N, K) > limit
    fake = 0x1000  # never dereferenced: the size check comes first
    assert L.bitlinear_forward_static(fake, fake, fake, M, K, N, fake, None) == B.ERR_WORKSPACE
    assert L.bitlinear_forward_static(fake, fake, fake, 1, 24, 16, fake, None) == B.ERR_SHAPE
    # the argument checks come before the device is asked for the scratch's address
    assert L.bitlinear_forward_static(None, fake, fake, 1, 16, 16, fake, None) == B.ERR_ARG
    assert L.bitlinear_forward_static(fake, fake, fake + 2, 1, 16, 16, fake, None) == B.ERR_ALIGN
