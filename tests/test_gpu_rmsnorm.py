"""GPU parity of the RMSNorm in front of the activation quantiser (and of the forward that uses it) against the
CPU oracle: int8 codes, beta bits and row sums bit-exact; bf16 outputs within 1e-2 relative / 1e-3 absolute and,
since both sides fix the same operation order, expected bit-identical.  All calls go through the C ABI."""
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


def gain_vector(K, seed):
    g = torch.Generator().manual_seed(1000 + seed)
    return (1.0 + 0.1 * torch.randn(K, generator=g)).to(torch.float32)


def timing_oracle():
    from oracle import load_oracle
    return load_oracle("timing")  # same source as the parity build (pinned equal on the CPU), with OpenMP


@pytest.mark.parametrize("M,K,seed,frac,scale,eps_n", [
    (1, 16, 1, 0.0, 1.0, 1e-5), (3, 144, 2, 0.02, 20.0, 0.0), (8, 1536, 3, 0.01, 20.0, 1e-5), (5, 3200, 4, 0.0, 1.0, 1e-6),
    (2, 4096, 5, 0.005, 30.0, 1e-5), (4, 28672, 6, 0.005, 30.0, 1e-5), (130, 1024, 7, 0.01, 10.0, 1e-5),
    (1, 131072, 8, 0.0, 1.0, 1e-5)])
def test_rmsnorm_quantiser_bit_exact(M, K, seed, frac, scale, eps_n):
    H = S.activations(M, K, seed, outlier_frac=frac, outlier_scale=scale)
    g = gain_vector(K, seed)
    q_ref, b_ref, s_ref = timing_oracle().rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), eps_n)
    Xq, beta, rowsum = B.rmsnorm_quantize_acts(H.cuda(), g.cuda(), eps_n)
    assert np.array_equal(Xq.cpu().numpy(), q_ref)
    assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
    assert np.array_equal(rowsum.cpu().numpy(), s_ref)


def test_rmsnorm_quantiser_special_tokens():
    """An all-zero token (beta at its floor, codes 0) next to ordinary ones; a token with an infinity is flagged
    with beta = NaN; unit gain and eps_n = 0 on a token of +-1 leave the plain quantiser's result."""
    K = 320
    H = S.activations(4, K, 9)
    H[1] = 0
    g = gain_vector(K, 9)
    q_ref, b_ref, s_ref = timing_oracle().rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), 1e-5)
    Xq, beta, rowsum = B.rmsnorm_quantize_acts(H.cuda(), g.cuda(), 1e-5)
    assert np.array_equal(Xq.cpu().numpy(), q_ref) and not Xq[1].any()
    assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
    assert np.array_equal(rowsum.cpu().numpy(), s_ref)
    H[2, 5] = float("inf")
    _, beta, _ = B.rmsnorm_quantize_acts(H.cuda(), g.cuda(), 1e-5)
    assert bool(torch.isnan(beta[2])) and not bool(torch.isnan(beta[[0, 1, 3]]).any())
    ones = (torch.randint(0, 2, (3, K), generator=torch.Generator().manual_seed(3)) * 2 - 1).to(torch.bfloat16)
    a = B.rmsnorm_quantize_acts(ones.cuda(), torch.ones(K, device="cuda"), 0.0)
    b = B.quantize_acts(ones.cuda())
    assert all(torch.equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("M,K,N,seed", [(1, 3200, 3200, 1), (8, 1536, 4096, 2), (16, 4096, 1040, 3), (40, 3200, 528, 4),
                                        (300, 1536, 1024, 5), (48, 8640, 272, 6)])
def test_forward_rmsnorm_matches_oracle(M, K, N, seed):
    """Every kernel behind the forward (weight-streaming for 1 to 16 tokens, tensor-core GEMM beyond, tiles cut along
    K for the last shape) with the normalising quantiser in front."""
    orc = timing_oracle()
    W = S.latent_weights(N, K, seed)
    H = S.activations(M, K, seed, outlier_frac=0.01, outlier_scale=20.0)
    g = gain_vector(K, seed)
    T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
    q_ref, b_ref, _ = orc.rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), 1e-5)
    Y_ref = orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref)
    packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
    ws = B.alloc_workspace(M, N, K)
    for _ in range(2):  # twice on one workspace
        Y = B.forward_rmsnorm(packed, gamma, H.cuda(), g.cuda(), 1e-5, N, workspace=ws)
        assert B.poll_status(ws) == 0
        y = torch_bf16_to_bits(Y)
        a = bf16_bits_to_float32(y).astype(np.float64)
        b = bf16_bits_to_float32(Y_ref).astype(np.float64)
        assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b))
        assert np.array_equal(y, Y_ref), "expected bit-identical bf16 outputs"


def test_rmsnorm_quantiser_extreme_scales():
    """Tokens of very small and very large values, subnormal bfloat16s, and a spread of 40 binades inside a token: the
    integer sum of squares is relative to the token's own largest exponent, so none of this loses exactness."""
    K = 1024
    H = S.activations(6, K, 11).float()
    H[0] *= 2.0 ** -110          # the largest exponent field is below 22
    H[1] *= 2.0 ** -125          # mostly subnormal bfloat16 values
    H[2] *= 2.0 ** 100
    H[3, 0], H[3, 1] = 2.0 ** 30, 2.0 ** -10
    H[4] = 0
    H[4, 7] = 2.0 ** -130        # a single subnormal value
    H = H.to(torch.bfloat16)
    g = gain_vector(K, 11)
    for eps_n in (0.0, 1e-5):
        q_ref, b_ref, s_ref = timing_oracle().rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), eps_n)
        Xq, beta, rowsum = B.rmsnorm_quantize_acts(H.cuda(), g.cuda(), eps_n)
        assert np.array_equal(Xq.cpu().numpy(), q_ref)
        assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
        assert np.array_equal(rowsum.cpu().numpy(), s_ref)


@pytest.mark.parametrize("M", [1, 5, 12, 40])
def test_sequence_with_rmsnorm_gains(M):
    """A decoder layer's seven projections in one sequence: q, k, v and gate, up read the normalised block input
    (they carry a gain), o and down are quantised as they are.  On the weight-streaming kernels (1, 5, 12 tokens) and
    on the table-driven GEMM (40 tokens); twice on one workspace."""
    orc = timing_oracle()
    shapes = S.decoder_layer_shapes(256, 704, kv_dim=64)
    normed = {"q", "k", "v", "gate", "up"}
    layers, gains, refs = [], [], []
    for mi, sh in enumerate(shapes):
        W = S.latent_weights(sh.N, sh.K, 80 + mi)
        H = S.activations(M, sh.K, 80 + mi, outlier_frac=0.02, outlier_scale=10.0)
        g = gain_vector(sh.K, 80 + mi) if sh.name in normed else None
        T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
        if g is not None:
            q_ref, b_ref, _ = orc.rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), 1e-6)
            refs.append(orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref))
        else:
            refs.append(orc.forward(T_ref, g_ref, torch_bf16_to_bits(H)))
        packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
        layers.append((packed, gamma, H.cuda(), torch.zeros((M, sh.N), dtype=torch.bfloat16, device="cuda"), sh.N))
        gains.append(g.cuda() if g is not None else None)
    assert any(g is None for g in gains) and any(g is not None for g in gains)
    seq = B.Sequence(layers, gains=gains, norm_eps=1e-6)
    for _ in range(2):
        for l in layers:
            l[3].zero_()
        seq.forward()
        torch.cuda.synchronize()
        assert B.poll_status(seq.workspace) == 0
        for l, ref in zip(layers, refs):
            assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
    seq.close()


def test_rmsnorm_entry_points_reject_bad_arguments():
    L = B.load_library()
    fake = 0x1000
    assert L.bitlinear_rmsnorm_quantize_acts(fake, None, 1e-5, 1, 16, fake, fake, fake, None) == B.ERR_ARG
    assert L.bitlinear_rmsnorm_quantize_acts(fake, fake, -1.0, 1, 16, fake, fake, fake, None) == B.ERR_ARG
    assert L.bitlinear_rmsnorm_quantize_acts(fake, fake + 4, 1e-5, 1, 16, fake, fake, fake, None) == B.ERR_ALIGN
    assert L.bitlinear_rmsnorm_quantize_acts(fake, fake, 1e-5, 1, 24, fake, fake, fake, None) == B.ERR_SHAPE
    assert L.bitlinear_forward_rmsnorm(fake, fake, fake, None, 1e-5, 1, 16, 16, fake, fake, 1 << 20, None) == B.ERR_ARG
