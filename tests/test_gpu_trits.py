"""GPU parity of the base-3 storage format (five weights per byte) against the CPU oracle.

Stored bytes, gamma bits, unpacked weights and int32 accumulators must be bit-exact; the bf16 outputs must be within
1e-2 relative / 1e-3 absolute and are expected to equal the oracle's bits, as on the 2-bit path (the arithmetic is the
same: only the stored bytes differ).  All calls go through the C ABI via the ctypes binding.
"""
import numpy as np
import pytest
import torch

from conftest import torch_bf16_to_bits
from oracle.oracle import bf16_bits_to_float32
from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu

REL_TOL, ABS_TOL = 1e-2, 1e-3


@pytest.fixture(scope="module")
def orc():
    from oracle import load_oracle
    from paper_2402_17764_b200 import build
    build.build()
    B.load_library()
    return load_oracle("timing")


def guarded(n, dtype, fill):
    pad = 256 // torch.empty(0, dtype=dtype).element_size()
    buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
    return buf, buf[pad:pad + n], pad


def guards_intact(buf, pad, n, fill):
    return bool((buf[:pad] == fill).all()) and bool((buf[pad + n:] == fill).all())


@pytest.mark.parametrize("N,K,seed,eps", [(16, 16, 0, 1e-5), (80, 64, 1, 1e-5), (96, 144, 2, 0.0), (3200, 3200, 3, 1e-5),
                                          (1024, 8640, 4, 1e-5), (16, 131072, 5, 1e-5), (4112, 80, 6, 1e-5)])
def test_quantize_weights_trits_bit_exact(orc, N, K, seed, eps):
    W = S.latent_weights(N, K, seed)
    T_ref, g_ref = orc.quantize_weights(W.numpy(), eps)
    p_ref = orc.pack_weights_trits(T_ref)
    nbytes = B.packed_bytes_trits(N, K)
    assert nbytes == p_ref.size
    buf, packed, pad = guarded(nbytes, torch.uint8, 0x5A)
    _, gamma = B.quantize_weights_trits(W.cuda(), eps, packed=packed)
    torch.cuda.synchronize()
    assert gamma.cpu().numpy().view(np.uint32)[0] == np.float32(g_ref).view(np.uint32), "gamma bits differ"
    assert np.array_equal(packed.cpu().numpy(), p_ref), "stored bytes differ"
    assert guards_intact(buf, pad, nbytes, 0x5A)
    assert np.array_equal(B.unpack_weights_trits(packed, N, K).cpu().numpy(), T_ref)
    assert int(packed.max()) <= 242


def test_quantize_weights_trits_hand_cases(golden):
    lay = golden["layout_trits"]
    N, K = lay["N"], lay["K"]
    for c in lay["cases"]:
        W = torch.zeros((N, K))
        W[c["n"], c["k"]] = float(c["t"])      # gamma = 1 / (N K): the one weight quantises to t, the rest to 0
        packed, _ = B.quantize_weights_trits(W.cuda(), 0.0)
        p = packed.cpu().numpy()
        assert np.nonzero(p != 121)[0].tolist() == [c["byte_index"]], c
        assert int(p[c["byte_index"]]) == c["byte_value"], c


@pytest.mark.parametrize("M,K,N", [(1, 16, 16), (1, 1536, 4096), (8, 1536, 4096), (3, 144, 96), (5, 8640, 1024), (1, 8192, 16),
                                   (2, 131072, 32), (7, 3200, 3200), (4, 80, 4112)])
def test_matmul_i32_trits(orc, M, K, N):
    rng = np.random.default_rng(M + K + N)
    T = rng.integers(-1, 2, (N, K)).astype(np.int8)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    packed = torch.from_numpy(orc.pack_weights_trits(T)).cuda()
    ref = orc.matmul_i32(Xq, T)
    buf, acc, pad = guarded(M * N, torch.int32, 23130)
    ws = B.alloc_workspace(M, N, K)
    L = B.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(2):  # twice on one workspace: the scratch must come back clean
        acc.fill_(-1)
        st = L.bitlinear_matmul_i32_trits(packed.data_ptr(), torch.from_numpy(Xq).cuda().data_ptr(), M, K, N, acc.data_ptr(),
                                          ws.data_ptr(), ws.numel(), stream)
        assert st == 0
        torch.cuda.synchronize()
        assert np.array_equal(acc.view(M, N).cpu().numpy(), ref)
        assert guards_intact(buf, pad, M * N, 23130)
        assert B.poll_status(ws) == 0


@pytest.mark.parametrize("M,K,N,seed", [(1, 3200, 3200, 1), (1, 8640, 3200, 2), (4, 4096, 11008, 3), (8, 11008, 4096, 4),
                                        (1, 16, 16, 5), (7, 144, 48, 6), (1, 16, 1 << 18, 7)])
def test_forward_trits(orc, M, K, N, seed):
    W = S.latent_weights(N, K, seed)
    X = S.activations(M, K, seed, outlier_frac=0.005, outlier_scale=30.0)
    T_ref, g_ref = orc.quantize_weights(W.numpy())
    want = orc.forward(T_ref, g_ref, torch_bf16_to_bits(X))
    packed, gamma = B.quantize_weights_trits(W.cuda())
    buf, Y, pad = guarded(M * N, torch.bfloat16, 23130)
    ws = B.alloc_workspace(M, N, K)
    B.forward_trits(packed, gamma, X.cuda(), N, Y=Y.view(M, N), workspace=ws)
    assert B.poll_status(ws) == 0
    got = torch_bf16_to_bits(Y.view(M, N))
    a, b = bf16_bits_to_float32(got).astype(np.float64), bf16_bits_to_float32(want).astype(np.float64)
    assert np.all(np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b))
    assert np.array_equal(got, want), "expected bit-identical bf16 outputs"
    assert guards_intact(buf, pad, M * N, 23130)
    # the 2-bit path gives the same bits
    p2, g2 = B.quantize_weights(W.cuda())
    assert torch.equal(B.forward(p2, g2, X.cuda(), N).view(torch.int16), Y.view(M, N).view(torch.int16))


def test_trits_sequence_and_limits(orc):
    """A small decoder layer set through one sequence on base-3 weights (twice: the workspace is reusable), and the
    limit of eight tokens."""
    for M in (1, 5):
        shapes = S.decoder_layer_shapes(256, 704, kv_dim=64)
        layers, refs = [], []
        for li in range(2):
            for mi, sh in enumerate(shapes):
                seed = li * 16 + mi
                W = S.latent_weights(sh.N, sh.K, seed)
                X = S.activations(M, sh.K, seed)
                T_ref, g_ref = orc.quantize_weights(W.numpy())
                refs.append(orc.forward(T_ref, g_ref, torch_bf16_to_bits(X)))
                packed, gamma = B.quantize_weights_trits(W.cuda())
                layers.append((packed, gamma, X.cuda(), torch.zeros((M, sh.N), dtype=torch.bfloat16, device="cuda"), sh.N))
        seq = B.Sequence(layers, trits=True)
        for _ in range(2):
            for l in layers:
                l[3].zero_()
            seq.forward()
            torch.cuda.synchronize()
            assert B.poll_status(seq.workspace) == 0
            for l, ref in zip(layers, refs):
                assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
        seq.close()
    W = S.latent_weights(16, 16, 0).cuda()
    packed, gamma = B.quantize_weights_trits(W)
    with pytest.raises(B.BitLinearError) as e:
        B.forward_trits(packed, gamma, S.activations(9, 16, 0).cuda(), 16)
    assert e.value.status == B.ERR_SHAPE


def test_3b_decode_step_trits_sampled(orc):
    """The 3B-shaped step (182 matrices, M = 1) on base-3 weights, as the benchmark runs it: sampled outputs of chosen
    matrices against the oracle, and 4/5 of the 2-bit bytes."""
    cfg = S.CONFIGS["3b_decode"]
    layers, meta, nbytes = [], [], 0
    for li in range(cfg["n_layers"]):
        for mi, sh in enumerate(cfg["layers"]):
            seed = li * 16 + mi
            W = S.latent_weights(sh.N, sh.K, seed, device="cuda")
            packed, gamma = B.quantize_weights_trits(W)
            del W
            X = S.activations(1, sh.K, seed, device="cuda")
            layers.append((packed, gamma, X, torch.zeros((1, sh.N), dtype=torch.bfloat16, device="cuda"), sh.N))
            meta.append((seed, sh))
            nbytes += packed.numel()
    assert nbytes == sum(B.packed_bytes_trits(sh.N, sh.K) for _, sh in meta)
    assert abs(nbytes / (805376000 * 0.8) - 1.0) < 0.01
    seq = B.Sequence(layers, trits=True)
    for _ in range(2):
        for l in layers:
            l[3].zero_()
        seq.forward()
    torch.cuda.synchronize()
    assert B.poll_status(seq.workspace) == 0
    rng = np.random.default_rng(3)
    for i in [0, 4, 6, 7 * 12 + 5, 7 * 25 + 6]:
        seed, sh = meta[i]
        packed, gamma, X, Y, N = layers[i]
        W = S.latent_weights(sh.N, sh.K, seed, device="cuda").cpu().numpy()
        rows = np.sort(rng.choice(sh.N, size=96, replace=False))
        rows[0], rows[-1] = 0, sh.N - 1
        T, g = orc.quantize_weights(W)
        q, beta, _ = orc.quantize_acts(torch_bf16_to_bits(X))
        want = orc.dequant(orc.matmul_i32(q, np.ascontiguousarray(T[rows])), beta, g)
        got = torch_bf16_to_bits(Y[:, torch.as_tensor(rows, device="cuda")])
        assert np.array_equal(got, want), f"matrix {i}"
    for l in layers:
        assert bool((l[3] != 0).any())
    seq.close()
