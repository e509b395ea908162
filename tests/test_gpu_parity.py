"""GPU parity: every kernel of the CUDA library against the CPU oracle on the same seeded inputs.

Integer results (packed weights, gamma bits, int8 activations, beta bits, row sums, int32
accumulators) must be bit-exact.  bf16 outputs must be within 1e-2 relative / 1e-3 absolute
(the tolerance the benchmark definition states); they are expected to be bit-identical because
both sides use the same single-rounding fp32 formula, and the tests record that too.
All calls go through the C ABI via the ctypes binding.
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


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2402_17764_b200 import build
    build.build()
    B.load_library()
    assert torch.cuda.is_available()
    yield
    torch.cuda.synchronize()


def dev(t):
    return t.to("cuda")


def assert_bf16_close(y_gpu_bits, y_ref_bits, what=""):
    a = bf16_bits_to_float32(y_gpu_bits).astype(np.float64)
    b = bf16_bits_to_float32(y_ref_bits).astype(np.float64)
    bad = np.abs(a - b) > (ABS_TOL + REL_TOL * np.abs(b))
    assert not bad.any(), f"{what}: {bad.sum()} outputs outside 1e-2 rel / 1e-3 abs"


def guarded(shape, dtype):
    """Output tensor inside a larger buffer whose borders hold a sentinel (stands in for a memory checker)."""
    n = int(np.prod(shape)) if len(shape) else 1
    item = torch.empty(0, dtype=dtype).element_size()
    pad = 256 // item
    buf = torch.full((n + 2 * pad,), 0x5A if dtype in (torch.int8, torch.uint8) else 23130, dtype=dtype, device="cuda")
    view = buf[pad:pad + n].view(*shape) if n else buf[pad:pad].view(*shape)
    return buf, view, pad


def check_guards(buf, pad, n):
    head = buf[:pad].cpu()
    tail = buf[pad + n:].cpu()
    sentinel = head[0].item()
    assert bool((head == sentinel).all()) and bool((tail == sentinel).all()), "write outside the output buffer"


# ------------------------------------------------------------------ (a) weight quantiser / packer

@pytest.mark.parametrize("N,K,seed,eps", [
    (16, 16, 0, 1e-5), (32, 144, 1, 1e-5), (4096, 1536, 0, 1e-5), (48, 8640, 2, 0.0), (1024, 3200, 3, 1e-5),
    (16, 131072, 4, 1e-5),
])
def test_quantize_weights_bit_exact(oracle, N, K, seed, eps):
    W = S.latent_weights(N, K, seed)
    T_ref, g_ref = oracle.quantize_weights(W.numpy(), eps)
    p_ref = oracle.pack_weights(T_ref)
    nbytes = B.packed_bytes(N, K)
    assert nbytes == p_ref.size
    buf, packed, pad = guarded((nbytes,), torch.uint8)
    _, gamma = B.quantize_weights(dev(W), eps, packed=packed)
    torch.cuda.synchronize()
    assert gamma.cpu().numpy().view(np.uint32)[0] == np.float32(g_ref).view(np.uint32), "gamma bits differ"
    assert np.array_equal(packed.cpu().numpy(), p_ref), "packed bytes differ"
    check_guards(buf, pad, nbytes)
    T_gpu = B.unpack_weights(packed, N, K).cpu().numpy()
    assert np.array_equal(T_gpu, T_ref)
    assert set(np.unique(T_gpu).tolist()) <= {-1, 0, 1}


def test_quantize_weights_hand_cases(oracle, golden):
    for case in golden["weights"]:
        block = np.array(case["W"], np.float32)          # 2 x 4
        W = np.tile(block, (8, 4))                        # 16 x 16: the mean of |W| is unchanged
        packed, gamma = B.quantize_weights(dev(torch.from_numpy(W)), case["eps"])
        assert gamma.item() == case["gamma"], case["citation"]
        T = B.unpack_weights(packed, 16, 16).cpu().numpy()
        assert np.array_equal(T, np.tile(np.array(case["T"], np.int8), (8, 4))), case["citation"]


def test_quantize_weights_degenerate(oracle):
    W = torch.zeros(16, 32)
    for eps in (0.0, 1e-5):
        packed, gamma = B.quantize_weights(dev(W), eps)
        assert gamma.item() == 0.0
        assert np.array_equal(packed.cpu().numpy(), oracle.pack_weights(oracle.quantize_weights(W.numpy(), eps)[0]))
    W = S.latent_weights(16, 32, 0)
    W[3, 7] = float("inf")
    _, gamma = B.quantize_weights(dev(W))
    assert np.isnan(gamma.item()), "out-of-range weights are reported as gamma = NaN"
    # a matrix with large and tiny magnitudes: exercises both shift directions of the fixed-point sum
    W = S.latent_weights(32, 64, 5)
    W[0, :8] = torch.tensor([1e6, -3.5e5, 16777215.0, 1e-30, -1e-38, 1e-42, 0.0, -0.0])
    T_ref, g_ref = oracle.quantize_weights(W.numpy())
    packed, gamma = B.quantize_weights(dev(W))
    assert gamma.cpu().numpy().view(np.uint32)[0] == np.float32(g_ref).view(np.uint32)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack_weights(T_ref))


def test_gaussian_statistics_on_gpu():
    """~31 % zeros and E[gamma] = sigma*sqrt(2/pi) on the first workload's weight shape."""
    W = S.latent_weights(4096, 1536, 0, device="cuda")
    packed, gamma = B.quantize_weights(W)
    T = B.unpack_weights(packed, 4096, 1536)
    zeros = (T == 0).float().mean().item()
    assert abs(zeros - 0.310064) < 1.2e-3
    assert abs(gamma.item() - 0.02 * (2 / np.pi) ** 0.5) < 5e-5


# ------------------------------------------------------------------ (b) activation quantiser

@pytest.mark.parametrize("M,K,seed,frac,scale", [
    (1, 16, 0, 0.0, 1.0), (3, 1536, 1, 0.0, 1.0), (8, 1536, 0, 0.01, 20.0), (5, 8640, 2, 0.005, 30.0),
    (2, 28672, 3, 0.0, 1.0), (1, 131072, 4, 0.0, 1.0), (300, 5120, 5, 0.0, 1.0),
])
def test_quantize_acts_bit_exact(oracle, M, K, seed, frac, scale):
    X = S.activations(M, K, seed, outlier_frac=frac, outlier_scale=scale)
    q_ref, b_ref, s_ref = oracle.quantize_acts(torch_bf16_to_bits(X))
    Xq, beta, rowsum = B.quantize_acts(dev(X))
    assert np.array_equal(Xq.cpu().numpy(), q_ref)
    assert np.array_equal(beta.cpu().numpy().view(np.uint32), b_ref.view(np.uint32))
    assert np.array_equal(rowsum.cpu().numpy(), s_ref)
    assert int(Xq.abs().max()) <= 127


def test_quantize_acts_hand_cases(golden):
    for case in golden["activations"]:
        x = np.zeros(16, np.float32)
        x[:len(case["x"])] = case["x"]
        X = torch.from_numpy(x).to(torch.bfloat16).view(1, 16)
        Xq, beta, rowsum = B.quantize_acts(dev(X))
        assert Xq.cpu().numpy()[0, :len(case["q"])].tolist() == case["q"], case["citation"]
        assert beta.item() == np.float32(case["beta"]), case["citation"]
        assert rowsum.item() == case["rowsum"], case["citation"]


def test_quantize_acts_mixed_zero_token(oracle):
    X = S.activations(4, 256, 9)
    X[2] = 0
    q_ref, b_ref, s_ref = oracle.quantize_acts(torch_bf16_to_bits(X))
    Xq, beta, rowsum = B.quantize_acts(dev(X))
    assert np.array_equal(Xq.cpu().numpy(), q_ref) and np.array_equal(beta.cpu().numpy(), b_ref)
    assert beta[2].item() == np.float32(1e-5) and int(Xq[2].abs().max()) == 0


# ------------------------------------------------------------------ (c), (d) integer matmul through each path

def make_operands(oracle, M, K, N, seed):
    rng = np.random.default_rng(seed)
    T = rng.integers(-1, 2, (N, K)).astype(np.int8)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    packed = torch.from_numpy(oracle.pack_weights(T)).cuda()
    return T, Xq, packed


MATMUL_SHAPES = [
    (1, 16, 16), (1, 1536, 4096), (8, 1536, 4096), (3, 144, 48), (5, 8640, 1024), (1, 8192, 16), (2, 131072, 32),
]


@pytest.mark.parametrize("M,K,N", MATMUL_SHAPES)
@pytest.mark.parametrize("path", [B.PATH_DP4A, B.PATH_MMA])
def test_matmul_i32_decode_paths(oracle, M, K, N, path):
    T, Xq, packed = make_operands(oracle, M, K, N, M + K + N)
    ref = oracle.matmul_i32(Xq, T)
    buf, acc, pad = guarded((M, N), torch.int32)
    ws = B.alloc_workspace(M, N, K)
    st = B.load_library().bitlinear_matmul_i32(packed.data_ptr(), torch.from_numpy(Xq).cuda().data_ptr(), M, K, N,
                                               acc.data_ptr(), path, ws.data_ptr(), ws.numel(),
                                               torch.cuda.current_stream().cuda_stream)
    assert st == 0
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), ref)
    check_guards(buf, pad, M * N)
    assert B.poll_status(ws) == 0


@pytest.mark.parametrize("M,K,N", [(16, 4096, 4096), (17, 8640, 1024), (33, 3200, 3200), (64, 1536, 4096),
                                   (9, 144, 48), (20, 16, 16), (40, 3200, 1040), (64, 32768, 16), (12, 1024, 8256)])
def test_matmul_i32_mma_wider_batches(oracle, M, K, N):
    T, Xq, packed = make_operands(oracle, M, K, N, M * 7 + N)
    ref = oracle.matmul_i32(Xq, T)
    Xq_d = torch.from_numpy(Xq).cuda()
    acc = B.matmul_i32(packed, Xq_d, N, path=B.PATH_MMA)
    assert np.array_equal(acc.cpu().numpy(), ref)
    # run twice: the split-K scratch must be left clean and the result must not change
    ws = B.alloc_workspace(M, N, K)
    a1 = B.matmul_i32(packed, Xq_d, N, path=B.PATH_MMA, workspace=ws).clone()
    a2 = B.matmul_i32(packed, Xq_d, N, path=B.PATH_MMA, workspace=ws)
    assert torch.equal(a1, a2) and np.array_equal(a2.cpu().numpy(), ref)


TC_SHAPES = [(128, 128, 256), (1, 16, 16), (65, 3200, 320), (200, 8640, 528), (300, 1536, 1024), (512, 5120, 256),
             (64, 4096, 4096), (129, 144, 4112),
             (300, 8640, 272), (40, 16384, 1040),
             # few tiles and a long K: the CTAs take equal shares of the k blocks of all tiles, and tiles whose k blocks
             # lie in several shares are summed through the per-CTA slots (64-row stages, one token tile, two token tiles)
             (20, 32768, 2560), (100, 32768, 2576), (300, 20000, 2304),
             # at most half as many tiles as SMs: every tile is split along K among 2, 3 or 8 CTAs, each of which finishes
             # its share of the tile's outputs; ragged M, K and N; and one launch that still deals k-block shares
             (200, 2048, 6400), (512, 3200, 5120), (70, 2096, 528), (300, 4800, 12800)]


@pytest.mark.parametrize("M,K,N", TC_SHAPES)
def test_matmul_i32_tcgen05(oracle, M, K, N, path=B.PATH_TCGEN05):
    T, Xq, packed = make_operands(oracle, M, K, N, M + 3 * K + N)
    ref = load_timing_oracle().matmul_i32(Xq, T)
    buf, acc, pad = guarded((M, N), torch.int32)
    ws = B.alloc_workspace(M, N, K)
    st = B.load_library().bitlinear_matmul_i32(packed.data_ptr(), torch.from_numpy(Xq).cuda().data_ptr(), M, K, N,
                                               acc.data_ptr(), path, ws.data_ptr(), ws.numel(),
                                               torch.cuda.current_stream().cuda_stream)
    assert st == 0
    assert B.poll_status(ws) == 0, "a bounded wait expired inside the tensor-core kernel"
    got = acc.cpu().numpy()
    assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} accumulators differ"
    check_guards(buf, pad, M * N)


def load_timing_oracle():
    from oracle import load_oracle
    return load_oracle("timing")  # same source, -O3 -fopenmp; pinned equal to the parity build on CPU


def test_dispatch_consistency(oracle):
    """The same tokens through the streaming kernel and the tensor-core kernel give identical int32."""
    M, K, N = 40, 3200, 1024
    T, Xq, packed = make_operands(oracle, M, K, N, 77)
    Xq_d = torch.from_numpy(Xq).cuda()
    a = B.matmul_i32(packed, Xq_d, N, path=B.PATH_MMA)
    b = B.matmul_i32(packed, Xq_d, N, path=B.PATH_TCGEN05)
    c = B.matmul_i32(packed, Xq_d[:8].contiguous(), N, path=B.PATH_DP4A)
    assert torch.equal(a, b) and torch.equal(a[:8], c)
    one = B.matmul_i32(packed, Xq_d[5:6].contiguous(), N, path=B.PATH_MMA)
    assert torch.equal(one[0], a[5]), "row t of a batch equals the single-token run"


# ------------------------------------------------------------------ whole forward

def run_forward_case(oracle, M, K, N, seed, frac=0.0, scale=1.0, eps=1e-5, big=False):
    W = S.latent_weights(N, K, seed)
    X = S.activations(M, K, seed, outlier_frac=frac, outlier_scale=scale)
    orc = load_timing_oracle() if big else oracle
    T_ref, g_ref = orc.quantize_weights(W.numpy(), eps)
    Y_ref = orc.forward(T_ref, g_ref, torch_bf16_to_bits(X))
    packed, gamma = B.quantize_weights(dev(W), eps)
    buf, Y, pad = guarded((M, N), torch.bfloat16)
    ws = B.alloc_workspace(M, N, K)
    B.forward(packed, gamma, dev(X), N, Y=Y, workspace=ws)
    assert B.poll_status(ws) == 0
    y_bits = torch_bf16_to_bits(Y)
    assert_bf16_close(y_bits, Y_ref, f"forward M={M} K={K} N={N}")
    check_guards(buf, pad, M * N)
    return float((y_bits == Y_ref).mean())


def test_forward_first_workload(oracle):
    """M=8, K=1536, N=4096, N(0,0.02) weights, N(0,1) activations with 1 % of channels x20, seed 0."""
    same = run_forward_case(oracle, 8, 1536, 4096, 0, frac=0.01, scale=20.0)
    assert same == 1.0, "expected bit-identical bf16 outputs"


@pytest.mark.parametrize("M,K,N,seed", [(1, 3200, 3200, 1), (1, 8640, 3200, 2), (4, 4096, 11008, 3), (16, 11008, 4096, 4),
                                        (64, 4096, 4096, 5), (1, 16, 16, 6), (7, 144, 48, 7),
                                        # a million output features behind the smallest K (16384 row blocks of one
                                        # padded column tile), on the streaming kernel and on the GEMM
                                        (1, 16, 1 << 20, 8), (40, 16, 1 << 18, 9)])
def test_forward_decode_shapes(oracle, M, K, N, seed):
    same = run_forward_case(oracle, M, K, N, seed, frac=0.005, scale=30.0, big=True)
    assert same == 1.0


@pytest.mark.parametrize("M,K,N,seed", [(65, 1536, 512, 1), (300, 1536, 1024, 2), (512, 5120, 768, 3), (130, 8640, 272, 4),
                                        # 17 to 64 tokens: the GEMM on a tile of mostly absent rows, fewer than 32 of
                                        # them backed by spare workspace rows
                                        (17, 3200, 1040, 5), (31, 144, 4112, 6), (32, 1536, 512, 7), (48, 8640, 272, 8),
                                        # the largest K the library takes (accumulators up to 127 * 131072), smallest N
                                        (2, 131072, 16, 9), (40, 131072, 32, 10), (200, 131072, 16, 11),
                                        # the largest M the library takes
                                        (1 << 20, 16, 16, 12)])
def test_forward_prefill_shapes(oracle, M, K, N, seed):
    same = run_forward_case(oracle, M, K, N, seed, big=True)
    assert same == 1.0


def _ragged_shapes(seed, count, m_range):
    """Seeded shapes with ragged M, K and N (K and N multiples of 16, the library's rule)."""
    rng = np.random.default_rng(seed)
    return [(int(rng.integers(m_range[0], m_range[1] + 1)), 16 * int(rng.integers(1, 260)), 16 * int(rng.integers(1, 130)), 100 + i)
            for i in range(count)]


# (the last two: several CTA tiles per CTA, i.e. both accumulator buffers in turn and rings that wrap, with short tiles)
@pytest.mark.parametrize("M,K,N,seed", _ragged_shapes(17, 12, (17, 64)) + [(40, 1024, 65536, 200), (33, 256, 131072, 201)])
def test_forward_weight_stationary_kernel_ragged_shapes(oracle, M, K, N, seed):
    """17 to 64 tokens (MMAs of 32, 48 and 64 columns), K from one ragged k block to 32, N from one partly filled tile up."""
    same = run_forward_case(oracle, M, K, N, seed, frac=0.01, scale=20.0, big=True)
    assert same == 1.0


def test_forward_empty_batch_and_errors():
    W = S.latent_weights(16, 16, 0)
    packed, gamma = B.quantize_weights(dev(W))
    X = torch.empty((0, 16), dtype=torch.bfloat16, device="cuda")
    Y = B.forward(packed, gamma, X, 16, workspace=B.alloc_workspace(1, 16, 16))
    assert Y.shape == (0, 16)
    X1 = dev(S.activations(1, 16, 0))
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.BitLinearError) as e:
        B.forward(packed, gamma, X1, 16, workspace=small)
    assert e.value.status == B.ERR_WORKSPACE


def test_forward_is_deterministic(oracle):
    W = S.latent_weights(1024, 3200, 3)
    X = dev(S.activations(5, 3200, 3))
    packed, gamma = B.quantize_weights(dev(W))
    ws = B.alloc_workspace(5, 1024, 3200)
    y1 = B.forward(packed, gamma, X, 1024, workspace=ws).clone()
    y2 = B.forward(packed, gamma, X, 1024, workspace=ws)
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))


def test_tiles_cut_along_k_are_reusable():
    """Few tiles and a long K: the GEMM deals equal shares of the k blocks of all tiles, and the partial sums of tiles
    that lie in several shares travel through flags and per-CTA slots in the workspace.  The flags are cleared by every
    call, so the same workspace gives the same (oracle) result again and again: as single matmuls (the third one deals
    shares by itself), and as a sequence whose matmuls have different K (table-driven launch, shares across matmuls)."""
    oracle = load_timing_oracle()
    specs = [(40, 20000, 1280), (64, 32768, 1552), (300, 20000, 2304)]
    layers, refs = [], []
    for i, (M, K, N) in enumerate(specs):
        W = S.latent_weights(N, K, 60 + i)
        X = S.activations(M, K, 60 + i, outlier_frac=0.01, outlier_scale=20.0)
        T_ref, g_ref = oracle.quantize_weights(W.numpy())
        refs.append(oracle.forward(T_ref, g_ref, torch_bf16_to_bits(X)))
        packed, gamma = B.quantize_weights(dev(W))
        Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        layers.append((packed, gamma, dev(X), Y, N))
    for (packed, gamma, X, Y, N), ref, (M, K, _) in zip(layers, refs, specs):
        ws = B.alloc_workspace(M, N, K)
        for _ in range(3):
            Y.zero_()
            B.forward(packed, gamma, X, N, Y=Y, workspace=ws)
            assert B.poll_status(ws) == 0
            assert np.array_equal(torch_bf16_to_bits(Y), ref)
    for part in (layers[:2], layers):  # 64-row stages; two token tiles per CTA tile
        seq = B.Sequence(part)
        for _ in range(3):
            for l in part:
                l[3].zero_()
            seq.forward()
            torch.cuda.synchronize()
            assert B.poll_status(seq.workspace) == 0
            for l, ref in zip(part, refs):
                assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
        seq.close()


def test_forward_sequence_matches_single_calls(oracle):
    """A small decoder layer set (7 projections x 2 layers) at M = 1 and M = 5."""
    for M in (1, 5):
        shapes = S.decoder_layer_shapes(256, 704, kv_dim=64)
        layers, refs = [], []
        for li in range(2):
            for mi, sh in enumerate(shapes):
                seed = li * 16 + mi
                W = S.latent_weights(sh.N, sh.K, seed)
                X = S.activations(M, sh.K, seed)
                T_ref, g_ref = oracle.quantize_weights(W.numpy())
                refs.append(oracle.forward(T_ref, g_ref, torch_bf16_to_bits(X)))
                packed, gamma = B.quantize_weights(dev(W))
                Y = torch.zeros((M, sh.N), dtype=torch.bfloat16, device="cuda")
                layers.append((packed, gamma, dev(X), Y, sh.N))
        few = B.Sequence(layers[:3])  # short lists travel as kernel parameters, long ones through device memory
        few.forward()
        torch.cuda.synchronize()
        for l, ref in zip(layers[:3], refs[:3]):
            assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
        few.close()
        seq = B.Sequence(layers)
        for _ in range(2):  # twice: the workspace must be reusable
            for l in layers:
                l[3].zero_()
            seq.forward()
            torch.cuda.synchronize()
            assert B.poll_status(seq.workspace) == 0
            for l, ref in zip(layers, refs):
                assert np.array_equal(torch_bf16_to_bits(l[3]), ref)
        seq.close()


@pytest.mark.parametrize("specs", [
    # largest M in 9..16: the weight-streaming kernel in which the warps of a CTA share the activations
    [(3, 144, 48), (16, 1536, 1040), (1, 3200, 512), (12, 80, 528), (9, 8640, 16)],
    # largest M in 17..128: every matmul in one launch of the tensor-core GEMM, one token tile per CTA tile
    [(3, 144, 48), (20, 1536, 1040), (1, 3200, 512), (64, 80, 528), (9, 8640, 16)],
    # largest M above 128: the same with two token tiles per CTA tile; more entries than travel as kernel parameters
    [(3, 144, 48), (300, 1536, 1040), (1, 3200, 512), (129, 80, 528), (9, 8640, 16), (256, 272, 272), (40, 144, 4112),
     (7, 16, 16), (130, 1024, 320), (2, 4096, 256)],
], ids=["max16", "max64", "max300"])
def test_forward_sequence_with_mixed_token_counts(oracle, specs):
    """Entries of one sequence may have different M; the largest one decides which kernel runs the whole sequence.
    Ragged shapes: N and K not multiples of 64."""
    layers, refs = [], []
    for i, (M, K, N) in enumerate(specs):
        W = S.latent_weights(N, K, 40 + i)
        X = S.activations(M, K, 40 + i, outlier_frac=0.02, outlier_scale=10.0)
        T_ref, g_ref = oracle.quantize_weights(W.numpy())
        refs.append(oracle.forward(T_ref, g_ref, torch_bf16_to_bits(X)))
        packed, gamma = B.quantize_weights(dev(W))
        buf, Y, pad = guarded((M, N), torch.bfloat16)
        layers.append((packed, gamma, dev(X), Y, N))
        layers[-1] = layers[-1] + (buf, pad)
    seq = B.Sequence([l[:5] for l in layers])
    for _ in range(2):
        seq.forward()
        torch.cuda.synchronize()
        assert B.poll_status(seq.workspace) == 0
        for (packed, gamma, X, Y, N, buf, pad), ref in zip(layers, refs):
            assert np.array_equal(torch_bf16_to_bits(Y), ref)
            check_guards(buf, pad, Y.numel())
    seq.close()
