"""Second, independent statement of the oracle in Python/numpy for SMALL shapes.

TEST INFRASTRUCTURE ONLY.  It exists to cross-check oracle/bitlinear_oracle.c:
the steps are the same ones of Section 2 (Eq. 1-3 and the per-token activation
quantiser) but written with different tools (Python integers and fractions,
numpy float32 scalars) and, for the 2-bit storage, from the opposite
direction: the C code maps (row, column) to a storage position, this file
walks the storage positions and says which (row, column) each one holds.
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
    T = np.clip(np.rint(W / denom), -1, 1).astype(np.int8)
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
