"""GPU parity of the SwiGLU in front of the activation quantiser (and of the forward that uses it) against the CPU
oracle: int8 codes, beta bits and row sums bit-exact; bf16 outputs within 1e-2 relative / 1e-3 absolute and, since both
sides fix the same operation order, expected bit-identical.  All calls go through the C ABI."""
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
    return load_oracle("timing")  # same source as the parity build (pinned equal on the CPU), with OpenMP


def gate_and_up(M, K, seed, gate_scale=2.5, frac=0.01, scale=10.0):
    """Outputs of a gate and an up projection: Gaussian with a few outliers, the gate wide enough to reach both
    saturated ends of the sigmoid now and then."""
    gate = (S.activations(M, K, seed, outlier_frac=frac, outlier_scale=scale).float() * gate_scale).to(torch.bfloat16)
    up = S.activations(M, K, 7000 + seed, outlier_frac=frac, outlier_scale=scale)
    return gate, up


def check_quantiser(gate, up):
    q_ref, b_ref, s_ref = timing_oracle().swiglu_quantize_acts(torch_bf16_to_bits(gate), torch_bf16_to_bits(up))
    Xq, beta, rowsum = B.swiglu_quantize_acts(gate.cuda(), up.cuda())
    assert np.array_equal(Xq.cpu().numpy(), q_ref)
    assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
    assert np.array_equal(rowsum.cpu().numpy(), s_ref)
    return Xq, beta, rowsum


@pytest.mark.parametrize("M,K,seed,gate_scale", [
    (1, 16, 1, 1.0), (3, 144, 2, 2.5), (8, 1536, 3, 2.5), (5, 8640, 4, 1.0), (2, 11008, 5, 4.0), (4, 28672, 6, 2.5),
    (130, 1024, 7, 30.0), (1, 131072, 8, 2.5), (6, 8192 + 64, 9, 2.5)])
def test_swiglu_quantiser_bit_exact(M, K, seed, gate_scale):
    """Tokens shorter than, equal to and longer than what the threads keep in registers (8192 elements)."""
    gate, up = gate_and_up(M, K, seed, gate_scale)
    check_quantiser(gate, up)


def test_swiglu_quantiser_whole_gate_range():
    """Every bfloat16 gate from -100 to 100 (both saturated ends, the breakpoints at +-87, zeros, subnormals) against
    several up values."""
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    vals = bf16_bits_to_float32(bits)
    keep = np.isfinite(vals) & (np.abs(vals) <= 100.0)
    g = torch.from_numpy(vals[keep].copy()).to(torch.bfloat16)
    K = (g.numel() + 15) // 16 * 16
    gate = torch.zeros((4, K), dtype=torch.bfloat16)
    gate[:, :g.numel()] = g
    up = torch.ones((4, K), dtype=torch.bfloat16)
    up[1] = -3.0
    up[2] = S.activations(1, K, 5)[0]
    up[3] = 2.0 ** -20
    check_quantiser(gate, up)


def test_swiglu_quantiser_special_tokens():
    """Zero gates or zero ups give zero codes (beta at its floor); an infinity or a NaN in either input, or a product
    beyond fp32, flags the token with beta = NaN and leaves the others alone; a saturated gate 2^7 leaves the plain
    quantiser's codes of the up input."""
    K = 320
    gate, up = gate_and_up(6, K, 11)
    gate[1] = 0
    up[2] = 0
    Xq, beta, _ = check_quantiser(gate, up)
    assert not Xq[1].any() and not Xq[2].any() and float(beta[1]) == float(np.float32(1e-5))
    gate[0, 5] = float("inf")
    up[3, 7] = float("nan")
    gate[4, 9], up[4, 9] = 2.0 ** 100, 2.0 ** 100
    _, beta, _ = B.swiglu_quantize_acts(gate.cuda(), up.cuda())
    assert bool(torch.isnan(beta[[0, 3, 4]]).all()) and not bool(torch.isnan(beta[[1, 2, 5]]).any())
    sat = torch.full((3, K), 128.0, dtype=torch.bfloat16)
    plain = gate_and_up(3, K, 12)[1]
    a = B.swiglu_quantize_acts(sat.cuda(), plain.cuda())
    b = B.quantize_acts(plain.cuda())
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], 128.0 * b[1]) and torch.equal(a[2], b[2])


@pytest.mark.parametrize("M,K,N,seed", [(1, 8640, 3200, 1), (8, 1536, 4096, 2), (16, 11008, 1040, 3), (40, 3200, 528, 4),
                                        (300, 1536, 1024, 5), (48, 8640, 272, 6)])
def test_forward_swiglu_matches_oracle(M, K, N, seed):
    """Every kernel behind the forward (weight-streaming for 1 to 16 tokens, tensor-core GEMM beyond, tiles cut along
    K for the last shape) with the SwiGLU quantiser in front: the down projection of a feed-forward block."""
    orc = timing_oracle()
    W = S.latent_weights(N, K, seed)
    gate, up = gate_and_up(M, K, seed)
    T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
    q_ref, b_ref, _ = orc.swiglu_quantize_acts(torch_bf16_to_bits(gate), torch_bf16_to_bits(up))
    Y_ref = orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref)
    packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
    ws = B.alloc_workspace(M, N, K)
    for _ in range(2):  # twice on one workspace
        Y = B.forward_swiglu(packed, gamma, gate.cuda(), up.cuda(), N, workspace=ws)
        assert B.poll_status(ws) == 0
        y = torch_bf16_to_bits(Y)
        a = bf16_bits_to_float32(y).astype(np.float64)
        b = bf16_bits_to_float32(Y_ref).astype(np.float64)
        assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b))
        assert np.array_equal(y, Y_ref), "expected bit-identical bf16 outputs"


@pytest.mark.parametrize("M", [1, 12, 40])
def test_sequence_with_all_fronts(M):
    """A decoder layer's seven projections in one sequence: q, k, v and gate, up carry an RMSNorm gain, down takes a
    gate and an up input (SwiGLU), o is quantised as it is.  Twice on one workspace."""
    orc = timing_oracle()
    shapes = S.decoder_layer_shapes(256, 704, kv_dim=64)
    normed = {"q", "k", "v", "gate", "up"}
    layers, gains, ups, refs = [], [], [], []
    for mi, sh in enumerate(shapes):
        W = S.latent_weights(sh.N, sh.K, 90 + mi)
        T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
        g, u = None, None
        if sh.name == "down":
            H, u = gate_and_up(M, sh.K, 90 + mi)
            q_ref, b_ref, _ = orc.swiglu_quantize_acts(torch_bf16_to_bits(H), torch_bf16_to_bits(u))
            refs.append(orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref))
        else:
            H = S.activations(M, sh.K, 90 + mi, outlier_frac=0.02, outlier_scale=10.0)
            if sh.name in normed:
                g = (1.0 + 0.1 * torch.randn(sh.K, generator=torch.Generator().manual_seed(mi))).to(torch.float32)
                q_ref, b_ref, _ = orc.rmsnorm_quantize_acts(torch_bf16_to_bits(H), g.numpy(), 1e-6)
                refs.append(orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref))
            else:
                refs.append(orc.forward(T_ref, g_ref, torch_bf16_to_bits(H)))
        packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
        layers.append((packed, gamma, H.cuda(), torch.zeros((M, sh.N), dtype=torch.bfloat16, device="cuda"), sh.N))
        gains.append(g.cuda() if g is not None else None)
        ups.append(u.cuda() if u is not None else None)
    assert sum(u is not None for u in ups) == 1 and sum(g is not None for g in gains) == 5
    for use_gains in (gains, None):  # with the RMSNorm entries, and with SwiGLU as the only front
        if use_gains is None:
            keep = [i for i, g in enumerate(gains) if g is None]
            sub_layers, sub_ups, sub_refs = [layers[i] for i in keep], [ups[i] for i in keep], [refs[i] for i in keep]
        else:
            sub_layers, sub_ups, sub_refs = layers, ups, refs
        seq = B.Sequence(sub_layers, gains=use_gains, norm_eps=1e-6, ups=sub_ups)
        for _ in range(2):
            for l in sub_layers:
                l[3].zero_()
            seq.forward()
            torch.cuda.synchronize()
            assert B.poll_status(seq.workspace) == 0
            for l, ref in zip(sub_layers, sub_refs):
                assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
        seq.close()


def test_swiglu_entry_points_reject_bad_arguments():
    L = B.load_library()
    fake = 0x1000
    assert L.bitlinear_swiglu_quantize_acts(fake, None, 1, 16, fake, fake, fake, None) == B.ERR_ARG
    assert L.bitlinear_swiglu_quantize_acts(fake, fake + 4, 1, 16, fake, fake, fake, None) == B.ERR_ALIGN
    assert L.bitlinear_swiglu_quantize_acts(fake, fake, 1, 24, fake, fake, fake, None) == B.ERR_SHAPE
    assert L.bitlinear_forward_swiglu(fake, fake, fake, None, 1, 16, 16, fake, fake, 1 << 20, None) == B.ERR_ARG
    assert L.bitlinear_forward_swiglu(fake, fake, fake, fake + 2, 1, 16, 16, fake, fake, 1 << 20, None) == B.ERR_ALIGN
    import ctypes
    descs = (B.LayerDesc * 1)(B.LayerDesc(fake, fake, fake, fake, 1, 16, 16))
    both = (ctypes.c_void_p * 1)(fake)
    out = ctypes.c_void_p()
    assert L.bitlinear_sequence_create_swiglu(descs, both, both, 1e-5, 1, fake, 1 << 20, ctypes.byref(out)) == B.ERR_ARG
    assert L.bitlinear_sequence_create_swiglu(descs, None, None, 1e-5, 1, fake, 1 << 20, ctypes.byref(out)) == B.ERR_ARG


def test_swiglu_empty_and_smallest_inputs():
    """No tokens: nothing is launched and nothing is touched; one token of 16 features: the smallest shape."""
    gate = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    Xq, beta, rowsum = B.swiglu_quantize_acts(gate, gate.clone())
    assert Xq.shape == (0, 64) and beta.numel() == 0 and rowsum.numel() == 0
    W = S.latent_weights(16, 16, 1)
    packed, gamma = B.quantize_weights(W.cuda(), 1e-5)
    ws = B.alloc_workspace(1, 16, 16)
    guard = torch.full((3, 16), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = B.forward_swiglu(packed, gamma, gate[:, :16].contiguous(), gate[:, :16].contiguous(), 16, Y=guard[1:1], workspace=ws)
    assert Y.shape == (0, 16) and bool((guard == 7.0).all())
    g1, u1 = gate_and_up(1, 16, 3)
    orc = timing_oracle()
    T_ref, g_ref = orc.quantize_weights(W.numpy(), 1e-5)
    q_ref, b_ref, _ = orc.swiglu_quantize_acts(torch_bf16_to_bits(g1), torch_bf16_to_bits(u1))
    want = orc.dequant(orc.matmul_i32(q_ref, T_ref), b_ref, g_ref)
    got = B.forward_swiglu(packed, gamma, g1.cuda(), u1.cuda(), 16, Y=guard[1:2], workspace=ws)
    assert np.array_equal(torch_bf16_to_bits(got), want)
    assert bool((guard[0] == 7.0).all()) and bool((guard[2] == 7.0).all())  # the rows around the output are untouched
