"""Second, independent statement of the oracle in Python/numpy for SMALL shapes.

TEST INFRASTRUCTURE ONLY.  It exists to cross-check oracle/bitlinear_oracle.c:
the steps are the same ones of Section 2 (Eq. 1-3 and the per-token activation
quantiser) but written with different tools (Python integers and fractions,
numpy float32 scalars) and, for the 2-bit storage, from the opposite
direction: the C code maps (row, column) to a storage position, this file
walks the storage positions and says which (row, column) each one holds.

The parts the paper only names (Section 2, "LLaMA-alike Components": RMSNorm and
SwiGLU in front of the quantiser; Section 4: activations of fewer bits) are
stated here from their textbook definitions in EXACT rational arithmetic, each
fp32 step of the fixed recipe being "the exact result, rounded once to the
nearest fp32, ties to even" (f32_of_fraction).  In particular the RMSNorm's
mean square is the exactly rounded mean of the exact squares: the C oracle's
integer sum, which cuts every square off 30 bits below the largest one, is
checked against it.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

QB = 127
BETA_FLOOR = np.float32(1e-5)


def bf16_bits_to_f32(bits) -> np.ndarray:
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits_rne(x) -> np.ndarray:
    u = np.asarray(x, np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def absmean(W) -> np.float32:
    """Eq. 3 with each |W_ij| truncated to a multiple of 2^-64 and summed exactly."""
    W = np.asarray(W, np.float32)
    total = 0
    for v in W.ravel():
        total += int(Fraction(abs(float(v))) * (1 << 64))  # int() floors a non-negative Fraction
    hi, lo = divmod(total, 1 << 64)
    s = (float(hi) * 2.0**64 + float(lo)) * 2.0**-64  # int->float conversions round to nearest
    return np.float32(s / float(W.size))


def quantize_weights(W, eps=1e-5):
    """Eq. 1-2: RoundClip(W / (gamma + eps), -1, 1) with round-half-to-even."""
    W = np.asarray(W, np.float32)
    g = absmean(W)
    denom = np.float32(g + np.float32(eps))
    with np.errstate(invalid="ignore"):
        ratio = W / denom
    ratio = np.where(np.isnan(ratio), np.float32(0.0), ratio)  # 0 / 0 (all-zero matrix, eps = 0): the weight is 0
    T = np.clip(np.rint(ratio), -1, 1).astype(np.int8)
    return T, g


def quantize_acts(X_bits):
    X = bf16_bits_to_f32(X_bits)
    M, K = X.shape
    Xq = np.zeros((M, K), np.int8)
    beta = np.zeros(M, np.float32)
    rowsum = np.zeros(M, np.int32)
    for t in range(M):
        b = max(np.float32(np.max(np.abs(X[t]))), BETA_FLOOR)
        s = np.float32(QB) / np.float32(b)
        q = np.clip(np.rint(X[t] * s), -QB, QB)
        Xq[t] = q.astype(np.int8)
        beta[t] = b
        rowsum[t] = int(q.sum())
    return Xq, beta, rowsum


def matmul_i32(Xq, T):
    M, K = Xq.shape
    N = T.shape[0]
    acc = np.zeros((M, N), np.int32)
    for t in range(M):
        for n in range(N):
            acc[t, n] = sum(int(a) * int(b) for a, b in zip(Xq[t], T[n]))
    return acc


def dequant(acc, beta, gamma):
    gamma = np.float32(gamma)
    scale = (gamma * beta.astype(np.float32)) / np.float32(QB)
    y = acc.astype(np.float32) * scale[:, None]
    return f32_to_bf16_bits_rne(y)


def quantize_acts_bits(X_bits, bits: int):
    """The activation quantiser with Q_b = 2^(bits-1) - 1 (Section 4 expects 4 bits or fewer; 8 gives Section 2)."""
    assert 2 <= bits <= 8
    return _quantize_rows(bf16_bits_to_f32(X_bits), (1 << (bits - 1)) - 1)


def dequant_bits(acc, beta, gamma, bits: int):
    qb = np.float32((1 << (bits - 1)) - 1)
    scale = (np.float32(gamma) * beta.astype(np.float32)) / qb
    return f32_to_bf16_bits_rne(acc.astype(np.float32) * scale[:, None])


def _quantize_rows(X, qb: int):
    """beta = max(absmax, 1e-5), s = qb / beta (one division), code = clip(rint(x * s)) for fp32 rows X."""
    X = np.asarray(X, np.float32)
    M, K = X.shape
    Xq = np.zeros((M, K), np.int8)
    beta = np.zeros(M, np.float32)
    rowsum = np.zeros(M, np.int32)
    for t in range(M):
        b = max(np.float32(np.max(np.abs(X[t]))), BETA_FLOOR)
        s = np.float32(qb) / np.float32(b)
        q = np.clip(np.rint(X[t] * s), -qb, qb)
        Xq[t] = q.astype(np.int8)
        beta[t] = b
        rowsum[t] = int(q.sum())
    return Xq, beta, rowsum


# ---- exact rational arithmetic with one rounding per step ----

def f32_of_fraction(q: Fraction) -> np.float32:
    """The fp32 value nearest to the rational q, ties to even, found with integer arithmetic only."""
    if q == 0:
        return np.float32(0.0)
    negative = q < 0
    q = abs(q)
    e = q.numerator.bit_length() - q.denominator.bit_length()  # 2^(e-1) < q < 2^(e+1)
    if Fraction(2) ** e > q:
        e -= 1                                                  # now 2^e <= q < 2^(e+1)
    e = max(e, -126)                                            # below the normal range the spacing stays 2^-149
    unit = Fraction(2) ** (e - 23)
    n, rest = divmod(q, unit)                                   # q = n * unit + rest, n < 2^24
    n = int(n)
    if 2 * rest > unit or (2 * rest == unit and n % 2 == 1):
        n += 1
    value = Fraction(n) * unit
    if value >= Fraction(2) ** 128:
        return np.float32(-np.inf if negative else np.inf)
    out = np.float32(float(value))                              # exact: value is an fp32 number
    return -out if negative else out


def _fr(x) -> Fraction:
    return Fraction(float(x))  # exact: every float is a rational


def _fma(a, b, c) -> np.float32:
    return f32_of_fraction(_fr(a) * _fr(b) + _fr(c))


def _mul(a, b) -> np.float32:
    return f32_of_fraction(_fr(a) * _fr(b))


def _add(a, b) -> np.float32:
    return f32_of_fraction(_fr(a) + _fr(b))


def _div(a, b) -> np.float32:
    return f32_of_fraction(_fr(a) / _fr(b))


def _sqrt(a) -> np.float32:
    """Correctly rounded square root of a non-negative fp32: the candidate whose neighbours' midpoints bracket a."""
    a = np.float32(a)
    if a == 0:
        return np.float32(0.0)
    c = np.float32(np.sqrt(np.float64(a)))
    fa = _fr(a)
    for cand in (np.nextafter(c, np.float32(0)), c, np.nextafter(c, np.float32(np.inf))):
        lo = (_fr(np.nextafter(cand, np.float32(0))) + _fr(cand)) / 2
        hi = (_fr(cand) + _fr(np.nextafter(cand, np.float32(np.inf)))) / 2
        if lo * lo <= fa <= hi * hi:  # (a tie cannot occur: a midpoint's square has too many bits to be an fp32)
            return np.float32(cand)
    raise AssertionError("no candidate brackets the square root")


def rmsnorm_mean_square(H_bits) -> np.ndarray:
    """mean_k h_k^2 of every token: the EXACT rational mean of the exact squares, rounded once to fp32."""
    H = bf16_bits_to_f32(H_bits)
    out = np.zeros(H.shape[0], np.float32)
    for t in range(H.shape[0]):
        total = sum((_fr(v) ** 2 for v in H[t]), Fraction(0))
        out[t] = f32_of_fraction(total / H.shape[1])
    return out


def rmsnorm_quantize_acts(H_bits, gain, eps_n):
    """x_k = h_k / sqrt(mean h^2 + eps_n) * g_k in the fixed fp32 steps (one rounding each: add, square root,
    reciprocal, two products), then the quantiser.  -> (Xq, beta, rowsum, x)."""
    H = bf16_bits_to_f32(H_bits)
    gain = np.asarray(gain, np.float32)
    M, K = H.shape
    mean = rmsnorm_mean_square(H_bits)
    x = np.zeros((M, K), np.float32)
    tiny = np.float32(2.0 ** -126)
    for t in range(M):
        d = _add(mean[t], np.float32(eps_n))
        if not d > tiny:
            d = tiny
        r = _div(np.float32(1.0), _sqrt(d))
        for k in range(K):
            x[t, k] = _mul(_mul(H[t, k], r), gain[k])
    return (*_quantize_rows(x, QB), x)


_LOG2E = np.float32(1.44269502162933349609375)
_LN2_HI = np.float32(0.693145751953125)
_LN2_LO = np.float32(1.42860676533018704503775e-06)
_TAYLOR = [Fraction(1, f) for f in (5040, 720, 120, 24, 6, 2, 1, 1)]  # 1/7!, 1/6!, ..., 1/1!, 1/0!


def sigmoid_f32(g) -> np.float32:
    """1 / (1 + e^-g) by the fixed recipe: range reduction by ln 2 in two parts, Taylor polynomial of degree 7."""
    t = -np.float32(g)
    if t > 87:
        return np.float32(0.0)
    if t < -87:
        return np.float32(1.0)
    z = _mul(t, _LOG2E)
    n = np.float32(np.rint(z))                                   # ties to even
    r = _fma(n, -_LN2_HI, t)
    r = _fma(n, -_LN2_LO, r)
    coeff = [f32_of_fraction(c) for c in _TAYLOR]                # the fp32 constants 1/5040.0f, ...
    p = _fma(r, coeff[0], coeff[1])
    for c in coeff[2:]:
        p = _fma(p, r, c)
    e = f32_of_fraction(_fr(p) * Fraction(2) ** int(n))          # exact scaling
    return _div(np.float32(1.0), _add(np.float32(1.0), e))


def swiglu_quantize_acts(G_bits, U_bits):
    """h_k = (g_k * sigmoid(g_k)) * u_k, then the quantiser.  -> (Xq, beta, rowsum, h)."""
    G, U = bf16_bits_to_f32(G_bits), bf16_bits_to_f32(U_bits)
    M, K = G.shape
    h = np.zeros((M, K), np.float32)
    for t in range(M):
        for k in range(K):
            h[t, k] = _mul(_mul(G[t, k], sigmoid_f32(G[t, k])), U[t, k])
    return (*_quantize_rows(h, QB), h)


def pack_weights(T) -> np.ndarray:
    """Walk the storage: tile -> slab -> 16-byte slot -> word -> byte -> 2-bit field, and fetch the weight it holds."""
    T = np.asarray(T, np.int8)
    N, K = T.shape
    assert N % 16 == 0
    row_blocks, col_tiles = (N + 63) // 64, (K + 63) // 64
    out = np.zeros(row_blocks * col_tiles * 1024, np.uint8)
    at = 0
    for row_block in range(row_blocks):
        for col_tile in range(col_tiles):
            for slab in range(2):               # columns 8*slab .. 8*slab+7 of every 16-column group
                for slot in range(32):          # 32 slots of four words each
                    row_low, col_group = slot // 4, slot % 4
                    for word in range(4):       # word: row half = word % 2, column half = word // 2
                        for byte in range(4):
                            v = 0
                            for field in range(4):
                                n = 64 * row_block + 16 * field + 8 * (word % 2) + row_low
                                k = 64 * col_tile + 16 * col_group + 8 * slab + 4 * (word // 2) + byte
                                code = int(T[n, k]) + 1 if (n < N and k < K) else 1
                                v |= code << (2 * field)
                            out[at] = v
                            at += 1
    return out


def pack_weights_trits(T) -> np.ndarray:
    """The base-3 storage (five weights per byte), walked from the storage side like pack_weights: tile -> slab -> slot
    -> word -> byte -> base-3 digit, fetching the weight each digit holds.  Row blocks have 80 rows."""
    T = np.asarray(T, np.int8)
    N, K = T.shape
    assert N % 16 == 0
    row_blocks, col_tiles = (N + 79) // 80, (K + 63) // 64
    out = np.zeros(row_blocks * col_tiles * 1024, np.uint8)
    at = 0
    for row_block in range(row_blocks):
        for col_tile in range(col_tiles):
            for slab in range(2):
                for slot in range(32):
                    row_low, col_group = slot // 4, slot % 4
                    for word in range(4):
                        for byte in range(4):
                            v = 0
                            for digit in range(4, -1, -1):      # Horner: the last row group is the leading digit
                                n = 80 * row_block + 16 * digit + 8 * (word % 2) + row_low
                                k = 64 * col_tile + 16 * col_group + 8 * slab + 4 * (word // 2) + byte
                                code = int(T[n, k]) + 1 if (n < N and k < K) else 1
                                v = 3 * v + code
                            out[at] = v
                            at += 1
    return out
