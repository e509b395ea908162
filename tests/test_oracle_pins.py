"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible mistake in the oracle (wrong tie rule, eps dropped, transposed
operand, wrong scale, wrong storage position) makes at least one of them fail.
"""
import math

import numpy as np
import pytest

from conftest import f32_to_bf16_bits
from oracle import np_restatement as R
from oracle.oracle import bf16_bits_to_float32


def bits_to_f32(b):
    return bf16_bits_to_float32(b)


# ---------------------------------------------------------------- hand cases (Eq. 1-3, Section 2)

def test_hand_cases_weights(oracle, golden):
    for case in golden["weights"]:
        W = np.array(case["W"], np.float32)
        T, g = oracle.quantize_weights(W, case["eps"])
        assert g == np.float32(case["gamma"]), case["citation"]
        assert T.tolist() == case["T"], case["citation"]


def test_hand_cases_activations(oracle, golden):
    for case in golden["activations"]:
        x = f32_to_bf16_bits(np.array([case["x"]], np.float32))
        q, beta, rs = oracle.quantize_acts(x)
        assert q[0].tolist() == case["q"], case["citation"]
        assert beta[0] == np.float32(case["beta"]), case["citation"]
        assert int(rs[0]) == case["rowsum"], case["citation"]


def test_hand_cases_forward(oracle, golden):
    for case in golden["forward"]:
        T = np.array(case["T"], np.int8)
        x = f32_to_bf16_bits(np.array([case["x"]], np.float32))
        Y, acc, Xq, beta, rs = oracle.forward(T, case["gamma"], x, return_all=True)
        assert acc[0].tolist() == case["acc"], case["citation"]
        assert bits_to_f32(Y)[0].tolist() == case["y"], case["citation"]


def test_zero_token_gives_zero_output(oracle):
    T = np.array([[1, -1, 0, 1]] * 16, np.int8)
    x = np.zeros((1, 4), np.uint16)
    Y = oracle.forward(T, 0.3, x)
    assert np.all(bits_to_f32(Y) == 0.0)


def test_hand_cases_layout(oracle, golden):
    lay = golden["layout"]
    N, K = lay["N"], lay["K"]
    base = oracle.pack_weights(np.zeros((N, K), np.int8))
    assert base.size == lay["packed_bytes"] and np.all(base == 0x55)
    for c in lay["cases"]:
        T = np.zeros((N, K), np.int8)
        T[c["n"], c["k"]] = 1
        p = oracle.pack_weights(T)
        diff = np.nonzero(p != 0x55)[0]
        assert diff.tolist() == [c["byte_index"]], (c, lay["citation"])
        assert int(p[c["byte_index"]]) == c["byte_value"], c


# ---------------------------------------------------------------- value sets

@pytest.mark.parametrize("seed", [0, 1])
def test_value_sets(oracle, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((64, 320)) * 0.02).astype(np.float32)
    T, g = oracle.quantize_weights(W)
    assert set(np.unique(T).tolist()) <= {-1, 0, 1}
    p = oracle.pack_weights(T)
    codes = np.stack([(p >> s) & 3 for s in (0, 2, 4, 6)])
    assert codes.max() <= 2, "code 3 must never be stored"
    x = rng.standard_normal((5, 320)).astype(np.float32)
    xbits = ((x.view(np.uint32) >> 16).astype(np.uint16))  # truncation to bf16 is fine for a value-set check
    q, beta, rs = oracle.quantize_acts(xbits)
    assert q.min() >= -127 and q.max() <= 127
    assert np.all(np.abs(q).max(axis=1) == 127), "the absmax element of each token maps to +-127"
    assert np.array_equal(rs, q.astype(np.int64).sum(axis=1).astype(np.int32))
    xf = bits_to_f32(xbits)
    assert np.array_equal(beta, np.abs(xf).max(axis=1))


def test_padding_columns_hold_code_one(oracle):
    rng = np.random.default_rng(3)
    N, K = 32, 144  # stored as 64 rows x 192 columns
    T = rng.integers(-1, 2, (N, K)).astype(np.int8)
    p = oracle.pack_weights(T)
    assert p.size == 64 * 192 // 4
    Tfull = np.zeros((64, 192), np.int8)
    Tfull[:N, :K] = T
    assert np.array_equal(p, oracle.pack_weights(Tfull))


# ---------------------------------------------------------------- closed forms on Gaussian input

def test_gaussian_closed_forms(oracle):
    sigma = 0.02
    rng = np.random.default_rng(0)
    N, K = 1024, 1536
    W = (rng.standard_normal((N, K)) * sigma).astype(np.float32)
    T, g = oracle.quantize_weights(W)
    n = N * K
    # E|w| = sigma*sqrt(2/pi); std of the sample mean = sigma*sqrt(1-2/pi)/sqrt(n)
    expect_gamma = sigma * math.sqrt(2 / math.pi)
    assert abs(float(g) - expect_gamma) < 5 * sigma * math.sqrt(1 - 2 / math.pi) / math.sqrt(n)
    # t = 0  <=>  |w| < gamma/2
    p0 = math.erf(0.5 * math.sqrt(2 / math.pi) / math.sqrt(2))
    assert abs(p0 - 0.310064) < 1e-5
    tol = 4 * math.sqrt(0.25 / n) + 2e-4  # binomial noise + the sampling noise of gamma itself
    assert abs((T == 0).mean() - p0) < tol
    assert abs((T == 1).mean() - (1 - p0) / 2) < tol
    assert abs((T == -1).mean() - (1 - p0) / 2) < tol


# ---------------------------------------------------------------- textbook reductions

@pytest.mark.parametrize("M,K,N", [(1, 64, 16), (7, 200, 48), (33, 1536, 64)])
def test_matmul_equals_numpy(oracle, M, K, N):
    rng = np.random.default_rng(M * 1000 + K)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    T = rng.integers(-1, 2, (N, K)).astype(np.int8)
    acc = oracle.matmul_i32(Xq, T)
    ref = Xq.astype(np.int64) @ T.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), ref)
    # an asymmetric case: a transposed operand or swapped index cannot pass both checks
    assert acc.shape == (M, N)


def test_forward_close_to_double_precision_product(oracle):
    """y ~= sum_k (gamma*t_nk) * (q_tk*beta_t/127) evaluated in double."""
    rng = np.random.default_rng(11)
    M, K, N = 6, 96, 32
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    x = rng.standard_normal((M, K)).astype(np.float32)
    xbits = (x.view(np.uint32) >> 16).astype(np.uint16)
    T, g = oracle.quantize_weights(W)
    Y, acc, Xq, beta, rs = oracle.forward(T, g, xbits, return_all=True)
    Wd = float(g) * T.astype(np.float64)
    Xd = Xq.astype(np.float64) * beta.astype(np.float64)[:, None] / 127.0
    ref = Xd @ Wd.T
    got = bits_to_f32(Y).astype(np.float64)
    # bf16 rounding is at most half an ulp = 2^-8 relative; the fp32 scale (two roundings) and the
    # fp32 product add a few 2^-24
    assert np.all(np.abs(got - ref) <= np.abs(ref) * (2.0**-8 + 2.0**-20) + 1e-12)  # 1e-12: the double sum's own noise
    # and the quantised product tracks the unquantised one (sanity of the scales' direction)
    full = bits_to_f32(xbits).astype(np.float64) @ (float(g) * T.astype(np.float64)).T
    assert np.corrcoef(full.ravel(), got.ravel())[0, 1] > 0.999


# ---------------------------------------------------------------- invariants

def test_invariants_weights(oracle):
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((32, 256)) * 0.02).astype(np.float32)
    T, g = oracle.quantize_weights(W, 0.0)
    Tn, gn = oracle.quantize_weights(-W, 0.0)
    assert gn == g and np.array_equal(Tn, -T)
    for j in (-3, 2, 7):
        Ts, gs = oracle.quantize_weights(np.ldexp(W, j), 0.0)
        assert gs == np.ldexp(g, j) and np.array_equal(Ts, T)
    # permuting entries leaves gamma unchanged bit for bit (order-free sum)
    perm = rng.permutation(W.size)
    assert oracle.absmean(W.ravel()[perm].reshape(W.shape)) == g


def test_invariants_activations_and_product(oracle):
    rng = np.random.default_rng(6)
    M, K, N = 4, 128, 32
    x = rng.standard_normal((M, K)).astype(np.float32)
    xbits = (x.view(np.uint32) >> 16).astype(np.uint16)
    q, beta, rs = oracle.quantize_acts(xbits)
    xf = bits_to_f32(xbits)
    q2, beta2, _ = oracle.quantize_acts(f32_to_bf16_bits(np.ldexp(xf, 3)))
    assert np.array_equal(q2, q) and np.array_equal(beta2, np.ldexp(beta, 3))
    qn, betan, rsn = oracle.quantize_acts(f32_to_bf16_bits(-xf))
    assert np.array_equal(qn, -q) and np.array_equal(betan, beta) and np.array_equal(rsn, -rs)
    T = rng.integers(-1, 2, (N, K)).astype(np.int8)
    acc = oracle.matmul_i32(q, T)
    perm = rng.permutation(K)
    assert np.array_equal(oracle.matmul_i32(q[:, perm], T[:, perm]), acc)
    # a row of a batch equals the single-token run of that row
    for t in range(M):
        Yt = oracle.forward(T, 0.017, xbits[t:t + 1])
        assert np.array_equal(Yt[0], oracle.forward(T, 0.017, xbits)[t])
    # offset-code identity: sum_k (t+1)*q = acc + rowsum
    assert np.array_equal(oracle.matmul_i32(q, (T + 1).astype(np.int8)), acc + rs[:, None])


def test_pack_unpack_roundtrip(oracle):
    rng = np.random.default_rng(7)
    for N, K in [(16, 128), (48, 320), (16, 64), (32, 8640 // 8)]:
        T = rng.integers(-1, 2, (N, K)).astype(np.int8)
        p = oracle.pack_weights(T)
        assert p.size == oracle.packed_bytes(N, K)
        assert np.array_equal(oracle.unpack_weights(p, N, K), T)


# ---------------------------------------------------------------- exactness of gamma

def test_gamma_matches_exactly_rounded_sum(oracle):
    rng = np.random.default_rng(8)
    for i in range(120):
        N = 16 * int(rng.integers(1, 6))
        K = int(rng.integers(8, 400))
        scale = 10.0 ** rng.uniform(-4, 2)
        W = (rng.standard_normal((N, K)) * scale).astype(np.float32)
        g = oracle.absmean(W)
        exact = math.fsum(abs(float(v)) for v in W.ravel()) / W.size  # fsum is correctly rounded
        assert g == np.float32(exact), (i, N, K)


def test_gamma_large_matrix_against_float128_free_reference(oracle):
    """A bigger matrix: compare with an exact integer sum done another way (numpy int64 on scaled values)."""
    rng = np.random.default_rng(9)
    # values that are exact multiples of 2^-20 and < 4 in magnitude: the exact sum fits int64
    ints = rng.integers(-(1 << 22), 1 << 22, (512, 2048))
    W = (ints.astype(np.float64) * 2.0**-20).astype(np.float32)
    assert np.array_equal(W.astype(np.float64) * 2.0**20, ints)
    exact = int(np.abs(ints).sum())
    g = oracle.absmean(W)
    assert g == np.float32((exact / W.size) * 2.0**-20) or g == np.float32(exact * 2.0**-20 / W.size)


def test_rejects_out_of_range(oracle):
    W = np.ones((16, 16), np.float32)
    W[3, 3] = np.inf
    with pytest.raises(ValueError):
        oracle.quantize_weights(W)
    W[3, 3] = 2.0**24
    with pytest.raises(ValueError):
        oracle.quantize_weights(W)


# ---------------------------------------------------------------- second statement in Python

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_c_oracle_equals_python_restatement(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    N, K, M = 32, 136 + 8 * seed, 3
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    x = rng.standard_normal((M, K)).astype(np.float32) * (1 + 19 * (rng.random(K) < 0.02))
    xbits = R.f32_to_bf16_bits_rne(x.astype(np.float32))
    T, g = oracle.quantize_weights(W)
    T2, g2 = R.quantize_weights(W)
    assert g == g2 and np.array_equal(T, T2)
    assert np.array_equal(oracle.pack_weights(T), R.pack_weights(T))
    q, beta, rs = oracle.quantize_acts(xbits)
    q2, beta2, rs2 = R.quantize_acts(xbits)
    assert np.array_equal(q, q2) and np.array_equal(beta, beta2) and np.array_equal(rs, rs2)
    acc = oracle.matmul_i32(q, T)
    assert np.array_equal(acc, R.matmul_i32(q, T))
    assert np.array_equal(oracle.dequant(acc, beta, g), R.dequant(acc, beta, g))
    assert np.array_equal(oracle.forward(T, g, xbits), R.dequant(acc, beta, g))


def test_timing_build_equals_parity_build(oracle):
    from oracle import load_oracle
    fast = load_oracle("timing")
    rng = np.random.default_rng(42)
    N, K, M = 64, 512, 9
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    x = rng.standard_normal((M, K)).astype(np.float32)
    xbits = R.f32_to_bf16_bits_rne(x)
    T, g = oracle.quantize_weights(W)
    T2, g2 = fast.quantize_weights(W)
    assert g == g2 and np.array_equal(T, T2)
    assert np.array_equal(oracle.forward(T, g, xbits), fast.forward(T, g, xbits))
    # the fronts of the quantiser and the b-bit variant: the GPU tests compare against the timing build
    gain = (1.0 + 0.1 * rng.standard_normal(K)).astype(np.float32)
    ubits = R.f32_to_bf16_bits_rne(rng.standard_normal((M, K)).astype(np.float32))
    gbits = R.f32_to_bf16_bits_rne((3.0 * rng.standard_normal((M, K))).astype(np.float32))
    for a, b in zip(oracle.rmsnorm_quantize_acts(xbits, gain, 1e-5, return_x=True),
                    fast.rmsnorm_quantize_acts(xbits, gain, 1e-5, return_x=True)):
        assert np.array_equal(a, b)
    for a, b in zip(oracle.swiglu_quantize_acts(gbits, ubits, return_h=True), fast.swiglu_quantize_acts(gbits, ubits, return_h=True)):
        assert np.array_equal(a, b)
    for a, b in zip(oracle.quantize_acts_bits(xbits, 4), fast.quantize_acts_bits(xbits, 4)):
        assert np.array_equal(a, b)
    acc = oracle.matmul_i32(oracle.quantize_acts_bits(xbits, 4)[0], T)
    beta = oracle.quantize_acts_bits(xbits, 4)[1]
    assert np.array_equal(oracle.dequant_bits(acc, beta, g, 4), fast.dequant_bits(acc, beta, g, 4))


# ---------------------------------------------------------------- RMSNorm in front of the quantiser

def _bf16(x):
    """bfloat16 bit patterns of x, the low 16 bits of each fp32 dropped (any bfloat16 input will do here)."""
    return (np.ascontiguousarray(x, np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_rmsnorm_quantiser_hand_case(oracle):
    """h = [3, 4, 0, -12], gain 1, eps_n 0: sum of squares 169, mean 42.25, rms 6.5 exactly; x = h / 6.5;
    beta = 12 / 6.5; x * 127 / beta = h * 127 / 12 = [31.75, 42.33, 0, -127] -> [32, 42, 0, -127]."""
    q, beta, rs, x = oracle.rmsnorm_quantize_acts(_bf16([[3, 4, 0, -12]]), np.ones(4, np.float32), 0.0, return_x=True)
    assert q.tolist() == [[32, 42, 0, -127]] and rs.tolist() == [-53]
    assert abs(float(beta[0]) - 12 / 6.5) < 2e-7 and np.allclose(x[0], np.array([3, 4, 0, -12]) / 6.5, rtol=3e-7, atol=0)
    # the gain multiplies after the normalisation: gain [2, 1, 1, 0.5] -> x = [6, 4, 0, -6] / 6.5, beta = 6 / 6.5
    q, beta, rs = oracle.rmsnorm_quantize_acts(_bf16([[3, 4, 0, -12]]), np.array([2, 1, 1, 0.5], np.float32), 0.0)
    assert q.tolist() == [[127, 85, 0, -127]] and rs.tolist() == [85]  # 4/6*127 = 84.67 -> 85
    # eps_n enters under the square root: mean 42.25 + 21.75 = 64 -> r = 1/8
    _, beta, _, x = oracle.rmsnorm_quantize_acts(_bf16([[3, 4, 0, -12]]), np.ones(4, np.float32), 21.75, return_x=True)
    assert x.tolist() == [[0.375, 0.5, 0.0, -1.5]] and beta.tolist() == [1.5]


def test_rmsnorm_matches_double_precision_and_library(oracle):
    import torch
    rng = np.random.default_rng(21)
    M, K, eps_n = 6, 1536, 1e-5
    h = rng.standard_normal((M, K)).astype(np.float32)
    h[:, rng.choice(K, 15, replace=False)] *= 20.0
    g = (1.0 + 0.1 * rng.standard_normal(K)).astype(np.float32)
    hb = _bf16(h)
    hf = bits_to_f32(hb).astype(np.float64)
    q, beta, rs, x = oracle.rmsnorm_quantize_acts(hb, g, eps_n, return_x=True)
    x64 = hf / np.sqrt((hf * hf).mean(axis=1, keepdims=True) + eps_n) * g.astype(np.float64)
    assert np.all(np.abs(x - x64) <= 4 * np.spacing(np.abs(x64).astype(np.float32)))      # a few fp32 roundings
    lib = torch.nn.functional.rms_norm(torch.from_numpy(hf), (K,), torch.from_numpy(g.astype(np.float64)), eps_n).numpy()
    assert np.allclose(x, lib, rtol=1e-6, atol=1e-9)
    b64 = np.abs(x64).max(axis=1)
    assert np.allclose(beta, b64, rtol=1e-6)
    scaled = x64 * (127.0 / b64)[:, None]
    clear = np.abs(scaled - np.floor(scaled) - 0.5) > 1e-3   # away from rounding ties, fp32 and fp64 must agree
    assert clear.mean() > 0.99 and np.array_equal(q[clear], np.rint(scaled)[clear].astype(np.int8))
    assert np.array_equal(rs, q.astype(np.int32).sum(axis=1)) and np.abs(q).max() == 127


def test_rmsnorm_quantiser_invariants(oracle):
    rng = np.random.default_rng(22)
    M, K = 5, 320
    hb = _bf16(rng.standard_normal((M, K)))
    g = (1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32)
    q, beta, rs = oracle.rmsnorm_quantize_acts(hb, g, 0.0)
    # without eps_n the scale of h cancels exactly (powers of two are exact in every step)
    q2, beta2, rs2 = oracle.rmsnorm_quantize_acts(_bf16(np.ldexp(bits_to_f32(hb), -5)), g, 0.0)
    assert np.array_equal(q2, q) and np.array_equal(beta2, beta) and np.array_equal(rs2, rs)
    # a permutation of the features (of h and the gain together) permutes the codes
    perm = rng.permutation(K)
    qp, betap, rsp = oracle.rmsnorm_quantize_acts(hb[:, perm], g[perm], 0.0)
    assert np.array_equal(qp, q[:, perm]) and np.array_equal(betap, beta) and np.array_equal(rsp, rs)
    # tokens with mean square exactly 1 and gain 1 are not changed by the normalisation: the plain quantiser
    ones = _bf16(rng.choice([-1.0, 1.0], size=(M, K)))
    qa, ba, ra = oracle.rmsnorm_quantize_acts(ones, np.ones(K, np.float32), 0.0)
    qb, bb, rb = oracle.quantize_acts(ones)
    assert np.array_equal(qa, qb) and np.array_equal(ba, bb) and np.array_equal(ra, rb)
    # an all-zero token gives zeros (beta at its floor), with or without eps_n
    for e in (0.0, 1e-5):
        qz, bz, rz = oracle.rmsnorm_quantize_acts(_bf16(np.zeros((1, K))), g, e)
        assert not qz.any() and rz[0] == 0
    # a huge spread inside a token: what lies more than 23 binades below the largest value adds nothing
    big = np.zeros((1, 16), np.float32)
    big[0, 0], big[0, 1] = 2.0 ** 30, 2.0 ** -10
    qs, bs, _ = oracle.rmsnorm_quantize_acts(_bf16(big), np.ones(16, np.float32), 0.0)
    assert qs[0, 0] == 127 and not qs[0, 1:].any() and bs[0] == 4.0   # x_0 = 2^30 / sqrt(2^60 / 16) = 4
    # infinities and NaNs are refused
    for v in (np.inf, np.nan):
        with pytest.raises(ValueError):
            oracle.rmsnorm_quantize_acts(_bf16([[v] + [0.0] * 15]), np.ones(16, np.float32), 0.0)


# ---- SwiGLU in front of the activation quantiser ----

def test_swiglu_quantiser_hand_cases(oracle):
    """g = 0: silu = 0.  Saturated gates: silu(g) = g for g > 87 and 0 for g < -87.  g = 1: 1 / (1 + 1/e)."""
    g = _bf16([[0.0, 128.0, -128.0, 1.0, -1.0, 96.0, 0.0, 0.0]])
    u = _bf16([[5.0, 0.5, 3.0, 2.0, 2.0, -1.0, 0.0, 0.0]])
    q, beta, rs, h = oracle.swiglu_quantize_acts(g, u, return_h=True)
    assert h[0, 0] == 0.0 and h[0, 1] == 64.0 and h[0, 2] == 0.0 and h[0, 5] == -96.0
    s1 = 1.0 / (1.0 + math.exp(-1.0))
    assert abs(float(h[0, 3]) - 2.0 * s1) < 3e-7 and abs(float(h[0, 4]) + 2.0 * (1.0 - s1)) < 3e-7
    assert beta.tolist() == [96.0]
    # 64 * 127 / 96 = 84.67, 2 * 0.7311 * 127 / 96 = 1.934, -2 * 0.2689 * 127 / 96 = -0.7115
    assert q.tolist() == [[0, 85, 0, 2, -1, -127, 0, 0]] and rs.tolist() == [-41]


def test_swiglu_matches_double_precision_and_library(oracle):
    import torch
    rng = np.random.default_rng(31)
    M, K = 6, 2048
    g = (2.5 * rng.standard_normal((M, K))).astype(np.float32)
    g[0, :64] = np.linspace(-87.0, 87.0, 64)          # the whole range of the exponential
    g[1, :64] = np.linspace(-20.0, 20.0, 64)
    u = rng.standard_normal((M, K)).astype(np.float32)
    gb, ub = _bf16(g), _bf16(u)
    g64, u64 = bits_to_f32(gb).astype(np.float64), bits_to_f32(ub).astype(np.float64)
    q, beta, rs, h = oracle.swiglu_quantize_acts(gb, ub, return_h=True)
    h64 = g64 / (1.0 + np.exp(-g64)) * u64
    # polynomial (below 1 ulp), the addition, the division and two products: a few fp32 roundings
    assert np.all(np.abs(h - h64) <= 6 * np.spacing(np.abs(h64).astype(np.float32)))
    lib = (torch.nn.functional.silu(torch.from_numpy(g64)) * torch.from_numpy(u64)).numpy()
    assert np.allclose(h, lib, rtol=1e-6, atol=1e-30)
    b64 = np.abs(h64).max(axis=1)
    assert np.allclose(beta, b64, rtol=1e-6)
    scaled = h64 * (127.0 / b64)[:, None]
    clear = np.abs(scaled - np.floor(scaled) - 0.5) > 1e-3   # away from rounding ties, fp32 and fp64 must agree
    assert clear.mean() > 0.99 and np.array_equal(q[clear], np.rint(scaled)[clear].astype(np.int8))
    assert np.array_equal(rs, q.astype(np.int32).sum(axis=1)) and np.abs(q).max() == 127


def test_swiglu_quantiser_invariants(oracle):
    rng = np.random.default_rng(32)
    M, K = 5, 320
    ub = _bf16(rng.standard_normal((M, K)))
    # a saturated gate 2^7 multiplies u by a power of two, which the quantiser does not see: the plain quantiser of u
    gate = _bf16(np.full((M, K), 128.0))
    q, beta, rs = oracle.swiglu_quantize_acts(gate, ub)
    qp, bp, rp = oracle.quantize_acts(ub)
    assert np.array_equal(q, qp) and np.array_equal(beta, 128.0 * bp) and np.array_equal(rs, rp)
    # odd in u; a permutation of the features permutes the codes
    gb = _bf16(3.0 * rng.standard_normal((M, K)))
    q, beta, rs = oracle.swiglu_quantize_acts(gb, ub)
    qn, bn, rn = oracle.swiglu_quantize_acts(gb, ub ^ np.uint16(0x8000))
    assert np.array_equal(qn, -q) and np.array_equal(bn, beta) and np.array_equal(rn, -rs)
    perm = rng.permutation(K)
    qq, bq, rq = oracle.swiglu_quantize_acts(gb[:, perm], ub[:, perm])
    assert np.array_equal(qq, q[:, perm]) and np.array_equal(bq, beta) and np.array_equal(rq, rs)
    # silu(g) - silu(-g) = g: the two halves of the sigmoid add up to one
    _, _, _, hp = oracle.swiglu_quantize_acts(gb, _bf16(np.ones((M, K))), return_h=True)
    _, _, _, hm = oracle.swiglu_quantize_acts(gb ^ np.uint16(0x8000), _bf16(np.ones((M, K))), return_h=True)
    gf = bits_to_f32(gb)
    assert np.all(np.abs((hp - hm) - gf) <= 4 * np.spacing(np.abs(gf)))
    # zero gates or zero ups give zeros (beta at its floor)
    for a, b in ((np.zeros((1, K)), rng.standard_normal((1, K))), (rng.standard_normal((1, K)), np.zeros((1, K)))):
        qz, bz, rz = oracle.swiglu_quantize_acts(_bf16(a), _bf16(b))
        assert not qz.any() and rz[0] == 0 and bz[0] == np.float32(1e-5)
    # infinities, NaNs and products beyond fp32 are refused
    for gv, uv in ((np.inf, 1.0), (1.0, np.nan), (-np.inf, 1.0), (2.0 ** 100, 2.0 ** 100)):
        with pytest.raises(ValueError):
            oracle.swiglu_quantize_acts(_bf16([[gv] + [0.0] * 15]), _bf16([[uv] + [1.0] * 15]))


# ---- activations of fewer bits ----

def test_low_bit_activations_hand_case(oracle):
    """b = 4: Q_b = 7.  A token with absmax 7 has s = 1: codes are the values rounded half to even."""
    x = _bf16([[7.0, 2.5, 3.5, -1.5, 0.5, -0.5, 6.5, -7.0, 0.25, 1.0, 0, 0, 0, 0, 0, 0]])
    q, beta, rs = oracle.quantize_acts_bits(x, 4)
    assert q.tolist() == [[7, 2, 4, -2, 0, 0, 6, -7, 0, 1, 0, 0, 0, 0, 0, 0]] and beta.tolist() == [7.0] and rs.tolist() == [11]
    # absmax 4: s = 1.75; 1 -> 1.75 -> 2, -2 -> -3.5 -> -4 (tie to even), 0.5 -> 0.875 -> 1, 0.25 -> 0.4375 -> 0
    q, beta, _ = oracle.quantize_acts_bits(_bf16([[1.0, -2.0, 0.5, 4.0, 0.25] + [0.0] * 11]), 4)
    assert q[0, :5].tolist() == [2, -4, 1, 7, 0] and beta.tolist() == [4.0]
    # b = 2: Q_b = 1, a sign with a dead zone below half the absmax
    q, _, _ = oracle.quantize_acts_bits(_bf16([[1.0, -0.75, 0.5, 0.25, -1.0] + [0.0] * 11]), 2)
    assert q[0, :5].tolist() == [1, -1, 0, 0, -1]
    # dequantisation: 14 * (0.5 * 2) / 7 = 2
    y = oracle.dequant_bits(np.array([[14, -7, 1]], np.int32), np.array([2.0], np.float32), 0.5, 4)
    assert bits_to_f32(y).tolist() == [[2.0, -1.0, float(bits_to_f32(_bf16([1.0 / 7.0]))[0])]]
    for bad in (1, 9):
        with pytest.raises(ValueError):
            oracle.quantize_acts_bits(x, bad)


def test_low_bit_activations_properties(oracle):
    rng = np.random.default_rng(41)
    M, K, N = 7, 640, 48
    xb = _bf16(rng.standard_normal((M, K)))
    xf = bits_to_f32(xb).astype(np.float64)
    # b = 8 is the quantiser of Section 2
    for a, b in zip(oracle.quantize_acts_bits(xb, 8), oracle.quantize_acts(xb)):
        assert np.array_equal(a, b)
    acc = rng.integers(-5000, 5000, (M, N)).astype(np.int32)
    beta8 = oracle.quantize_acts(xb)[1]
    assert np.array_equal(oracle.dequant_bits(acc, beta8, 0.02, 8), oracle.dequant(acc, beta8, 0.02))
    for bits in (2, 3, 4, 6):
        qb = 2 ** (bits - 1) - 1
        q, beta, rs = oracle.quantize_acts_bits(xb, bits)
        assert np.abs(q).max() == qb and np.array_equal(rs, q.astype(np.int32).sum(axis=1))
        assert np.array_equal(beta, np.abs(xf).max(axis=1).astype(np.float32))
        # each value is reproduced to within half a step
        err = np.abs(xf - q * (beta.astype(np.float64) / qb)[:, None])
        assert np.all(err <= (beta.astype(np.float64) / (2 * qb))[:, None] * (1 + 1e-6))
        # codes equal the double-precision ones away from ties
        scaled = xf * (qb / beta.astype(np.float64))[:, None]
        clear = np.abs(scaled - np.floor(scaled) - 0.5) > 1e-4
        assert clear.mean() > 0.99 and np.array_equal(q[clear], np.rint(scaled)[clear].astype(np.int8))
        # the forward is the double-precision product of the dequantised operands
        T = rng.integers(-1, 2, (N, K)).astype(np.int8)
        y = bits_to_f32(oracle.dequant_bits(oracle.matmul_i32(q, T), beta, 0.02, bits)).astype(np.float64)
        want = (q.astype(np.float64) * (beta.astype(np.float64) / qb)[:, None]) @ (T.astype(np.float64) * 0.02).T
        assert np.allclose(y, want, rtol=2.0 ** -8, atol=1e-9)


# ---- the all-zero matrix (0 / 0 in Eq. 1 when eps = 0) ----

def test_all_zero_matrix_quantises_to_zeros(oracle):
    """W = 0 and eps = 0: gamma = 0 and Eq. 1 divides 0 by 0.  Reading: every weight stays 0, so every stored field
    holds code 1 (byte 0b01010101) and the forward gives zeros; with eps > 0 the quotient is an ordinary 0."""
    W = np.zeros((16, 32), np.float32)
    for eps in (0.0, 1e-5):
        T, g = oracle.quantize_weights(W, eps)
        assert g == 0.0 and not T.any()
        assert np.all(oracle.pack_weights(T) == 0x55)
        assert np.array_equal(R.quantize_weights(W, eps)[0], T)
    xbits = f32_to_bf16_bits(np.arange(-16, 16, dtype=np.float32).reshape(1, 32))
    assert not oracle.forward(oracle.quantize_weights(W, 0.0)[0], 0.0, xbits).any()
    # a single non-zero weight among zeros is the only one that survives: gamma = 1/512, W/gamma = 512 -> clip 1
    W[3, 7] = -1.0
    T, g = oracle.quantize_weights(W, 0.0)
    assert g == np.float32(1.0 / 512.0) and T[3, 7] == -1 and np.abs(T).sum() == 1


# ---- second statements of the fronts and of the b-bit variant (exact rational arithmetic, one rounding per step) ----

def test_f32_of_fraction_is_round_to_nearest_even():
    from fractions import Fraction as F
    one = F(1)
    ulp = F(1, 2 ** 23)
    assert R.f32_of_fraction(one + ulp / 2) == np.float32(1.0)                  # tie -> even (1.0)
    assert R.f32_of_fraction(one + 3 * ulp / 2) == np.float32(1.0 + 2.0 ** -22)  # tie -> even (upwards)
    assert R.f32_of_fraction(one + ulp / 2 + F(1, 2 ** 80)) == np.float32(1.0 + 2.0 ** -23)
    assert R.f32_of_fraction(F(1, 3)) == np.float32(1.0 / 3.0) and R.f32_of_fraction(F(-1, 10)) == np.float32(-0.1)
    assert R.f32_of_fraction(F(1, 2 ** 149)) == np.float32(2.0 ** -149)          # smallest subnormal
    assert R.f32_of_fraction(F(1, 2 ** 150)) == 0.0 and R.f32_of_fraction(F(3, 2 ** 150)) == np.float32(2.0 ** -148)
    assert R.f32_of_fraction(F(2 ** 24 + 1)) == np.float32(2.0 ** 24) and np.isinf(R.f32_of_fraction(F(2) ** 128))
    rng = np.random.default_rng(5)
    for a, b in rng.standard_normal((200, 2)).astype(np.float32):               # numpy's IEEE operations agree
        assert R._mul(a, b) == a * b and R._add(a, b) == a + b and R._div(a, b) == a / b
        assert R._sqrt(abs(a)) == np.sqrt(np.float32(abs(a)))


def _token_mix(rng, M, K):
    """Tokens of several kinds: Gaussian, Gaussian with outlier channels, tiny and huge scales, a spread of many
    binades inside the token, subnormal magnitudes, a token of zeros with one value."""
    h = rng.standard_normal((M, K)).astype(np.float32)
    kind = np.arange(M) % 6
    h[kind == 1, : max(1, K // 64)] *= 30.0
    h[kind == 2] *= np.float32(2.0 ** -60)
    h[kind == 3] *= np.float32(2.0 ** 50)
    spread = np.ldexp(np.float32(1.0), rng.integers(-20, 21, size=(M, K)).astype(np.int32)).astype(np.float32)
    h[kind == 4] *= spread[kind == 4]
    h[kind == 5] *= np.float32(2.0 ** -120)
    return _bf16(h)


def test_rmsnorm_mean_square_is_the_exactly_rounded_mean_of_exact_squares(oracle):
    """The C oracle sums integers in which every square is cut off 30 bits below the largest one and divides in
    double.  The definition is the exact mean of the exact squares, rounded once.  On 1200 tokens of mixed kinds the two
    are the same fp32 number (they can differ only if the exact mean lies within a relative 2^-27 of a rounding
    boundary)."""
    rng = np.random.default_rng(77)
    checked = 0
    for K in (16, 48, 320, 1536):
        hb = _token_mix(rng, 300, K)
        got = oracle.rmsnorm_mean_square(hb)
        want = R.rmsnorm_mean_square(hb)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), f"K={K}: {(got != want).sum()} tokens differ"
        checked += len(got)
    assert checked >= 1000
    # powers of two: mean square of [2^a, 0, 0, 0] is 4^a / 4 exactly, over the whole exponent range of a bfloat16 square
    for a in (-60, -31, 0, 17, 60):
        hb = _bf16(np.array([[np.ldexp(1.0, a)] + [0.0] * 3], np.float32))
        assert float(oracle.rmsnorm_mean_square(hb)[0]) == np.ldexp(1.0, 2 * a - 2)


def test_c_oracle_equals_python_restatement_of_the_fronts(oracle):
    rng = np.random.default_rng(78)
    # RMSNorm: x, beta, codes and row sums bit for bit
    M, K = 24, 80
    hb = _token_mix(rng, M, K)
    gain = (1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32)
    for eps_n in (0.0, 1e-5):
        q, beta, rs, x = oracle.rmsnorm_quantize_acts(hb, gain, eps_n, return_x=True)
        q2, beta2, rs2, x2 = R.rmsnorm_quantize_acts(hb, gain, eps_n)
        assert np.array_equal(x.view(np.uint32), x2.view(np.uint32))
        assert np.array_equal(q, q2) and np.array_equal(beta, beta2) and np.array_equal(rs, rs2)
    # SwiGLU: gates over the whole range of the exponential, the saturated ends included
    M, K = 6, 96
    g = (4.0 * rng.standard_normal((M, K))).astype(np.float32)
    g[0] = np.linspace(-90.0, 90.0, K)
    g[1] = np.linspace(-1.0, 1.0, K)
    gb, ub = _bf16(g), _bf16(rng.standard_normal((M, K)))
    q, beta, rs, h = oracle.swiglu_quantize_acts(gb, ub, return_h=True)
    q2, beta2, rs2, h2 = R.swiglu_quantize_acts(gb, ub)
    assert np.array_equal(h.view(np.uint32), h2.view(np.uint32))
    assert np.array_equal(q, q2) and np.array_equal(beta, beta2) and np.array_equal(rs, rs2)
    # activations of fewer bits
    xb = _bf16(rng.standard_normal((5, 144)) * (1 + 19 * (rng.random(144) < 0.05)))
    acc = rng.integers(-20000, 20000, (5, 32)).astype(np.int32)
    for bits in (2, 3, 4, 5, 8):
        q, beta, rs = oracle.quantize_acts_bits(xb, bits)
        q2, beta2, rs2 = R.quantize_acts_bits(xb, bits)
        assert np.array_equal(q, q2) and np.array_equal(beta, beta2) and np.array_equal(rs, rs2)
        assert np.array_equal(oracle.dequant_bits(acc, beta, 0.0173, bits), R.dequant_bits(acc, beta, 0.0173, bits))


# ---- base-3 storage: five weights per byte ----

def test_hand_cases_layout_trits(oracle, golden):
    lay = golden["layout_trits"]
    N, K = lay["N"], lay["K"]
    base = oracle.pack_weights_trits(np.zeros((N, K), np.int8))
    assert base.size == lay["packed_bytes"] == oracle.packed_bytes_trits(N, K) and np.all(base == 121)
    for c in lay["cases"]:
        T = np.zeros((N, K), np.int8)
        T[c["n"], c["k"]] = c["t"]
        p = oracle.pack_weights_trits(T)
        diff = np.nonzero(p != 121)[0]
        assert diff.tolist() == [c["byte_index"]], (c, lay["citation"])
        assert int(p[c["byte_index"]]) == c["byte_value"], c


def test_trit_storage_properties(oracle):
    rng = np.random.default_rng(9)
    for N, K in [(16, 16), (80, 64), (96, 144), (176, 200), (3200, 320)]:
        T = rng.integers(-1, 2, (N, K)).astype(np.int8)
        p = oracle.pack_weights_trits(T)
        assert p.size == -(-N // 80) * -(-K // 64) * 1024      # 80 x 64 weights per KiB: 1.6 bits per weight
        assert p.max() <= 242                                    # 3^5 - 1: every byte is a five-digit base-3 number
        assert np.array_equal(oracle.unpack_weights_trits(p, N, K), T)
        if N * K <= 40000:
            assert np.array_equal(p, R.pack_weights_trits(T))
    # five weights per byte against four: the same matrix takes 4/5 of the bytes when N is a multiple of 80 and 64
    assert oracle.packed_bytes_trits(320, 640) * 5 == oracle.packed_bytes(320, 640) * 4
    # an all-ones matrix fills every digit with 2 (byte 242) where weights exist; minus ones give 0 there
    p = oracle.pack_weights_trits(np.ones((80, 64), np.int8))
    assert np.all(p == 242) and not oracle.pack_weights_trits(-np.ones((80, 64), np.int8)).any()
    with pytest.raises(ValueError):
        oracle.unpack_weights_trits(np.full(1024, 243, np.uint8), 80, 64)
