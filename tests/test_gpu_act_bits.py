"""GPU parity of the forward with activations of fewer than 8 bits against the CPU oracle: codes, beta bits and row
sums bit-exact, bf16 outputs within 1e-2 relative / 1e-3 absolute and expected bit-identical.  Through the C ABI."""
import numpy as np
import pytest
import torch

from conftest import torch_bf16_to_bits
from oracle.oracle import bf16_bits_to_float32
from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu

REL_TOL, ABS_TOL = 1e-2, 1e-3


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2402_17764_b200 import build
    build.build()
    B.load_library()
    assert torch.cuda.is_available()
    yield
    torch.cuda.synchronize()


def timing_oracle():
    from oracle import load_oracle
    return load_oracle("timing")


@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
@pytest.mark.parametrize("M,K,seed", [(1, 16, 1), (5, 3200, 2), (3, 11008, 3), (130, 1024, 4)])
def test_quantiser_bit_exact(bits, M, K, seed):
    X = S.activations(M, K, seed, outlier_frac=0.01, outlier_scale=20.0)
    q_ref, b_ref, s_ref = timing_oracle().quantize_acts_bits(torch_bf16_to_bits(X), bits)
    Xq, beta, rowsum = B.quantize_acts_bits(X.cuda(), bits)
    assert np.array_equal(Xq.cpu().numpy(), q_ref) and int(Xq.abs().max()) == 2 ** (bits - 1) - 1
    assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
    assert np.array_equal(rowsum.cpu().numpy(), s_ref)
    if bits == 8:
        for a, b in zip((Xq, beta, rowsum), B.quantize_acts(X.cuda())):
            assert torch.equal(a, b)


@pytest.mark.parametrize("bits", [4, 2])
@pytest.mark.parametrize("M,K,N,seed", [(1, 3200, 3200, 1), (8, 1536, 4096, 2), (16, 4096, 1040, 3), (40, 3200, 528, 4),
                                        (300, 1536, 1024, 5), (48, 8640, 272, 6)])
def test_forward_matches_oracle(bits, M, K, N, seed):
    """Every kernel behind the forward: weight-streaming for 1 to 16 tokens, tensor-core GEMM beyond (one and two token
    tiles; tiles cut along K for the last shape)."""
    orc = timing_oracle()
    W = S.latent_weights(N, K, seed)
    X = S.activations(M, K, seed, outlier_frac=0.01, outlier_scale=20.0)
    T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
    q_ref, b_ref, _ = orc.quantize_acts_bits(torch_bf16_to_bits(X), bits)
    Y_ref = orc.dequant_bits(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref, bits)
    packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
    ws = B.alloc_workspace(M, N, K)
    for _ in range(2):  # twice on one workspace
        Y = B.forward_act_bits(packed, gamma, X.cuda(), N, bits, workspace=ws)
        assert B.poll_status(ws) == 0
        y = torch_bf16_to_bits(Y)
        a = bf16_bits_to_float32(y).astype(np.float64)
        b = bf16_bits_to_float32(Y_ref).astype(np.float64)
        assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b))
        assert np.array_equal(y, Y_ref), "expected bit-identical bf16 outputs"
    # with 8 bits it is the forward of Section 2
    assert torch.equal(B.forward_act_bits(packed, gamma, X.cuda(), N, 8, workspace=ws).view(torch.int16),
                       B.forward(packed, gamma, X.cuda(), N, workspace=ws).view(torch.int16))


def test_entry_points_reject_bad_arguments():
    L = B.load_library()
    fake = 0x1000
    for bits in (1, 9, 0, -4):
        assert L.bitlinear_quantize_acts_bits(fake, 1, 16, bits, fake, fake, fake, None) == B.ERR_ARG
        assert L.bitlinear_forward_act_bits(fake, fake, fake, 1, 16, 16, bits, fake, fake, 1 << 20, None) == B.ERR_ARG
    assert L.bitlinear_quantize_acts_bits(fake, 1, 24, 4, fake, fake, fake, None) == B.ERR_SHAPE


def test_empty_input_and_guard_rows():
    X = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    Xq, beta, rowsum = B.quantize_acts_bits(X, 4)
    assert Xq.shape == (0, 64) and beta.numel() == 0 and rowsum.numel() == 0
    # a forward at 5 tokens writes its 5 rows of Y and nothing around them
    W = S.latent_weights(48, 80, 2)
    packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
    guard = torch.full((7, 48), -3.0, dtype=torch.bfloat16, device="cuda")
    x = S.activations(5, 80, 2)
    orc = timing_oracle()
    T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
    q_ref, b_ref, _ = orc.quantize_acts_bits(torch_bf16_to_bits(x), 4)
    want = orc.dequant_bits(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref, 4)
    got = B.forward_act_bits(packed, gamma, x.cuda(), 48, 4, Y=guard[1:6])
    assert np.array_equal(torch_bf16_to_bits(got), want)
    assert bool((guard[0] == -3.0).all()) and bool((guard[6] == -3.0).all())
