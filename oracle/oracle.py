"""ctypes front end of the C oracle (oracle/bitlinear_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  All arrays are numpy; bfloat16 travels as
uint16 bit patterns.  Two builds of the same source exist: "parity" (-O2, no
contraction, single thread) and "timing" (-O3 -fopenmp, outer loops parallel).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "bitlinear_oracle.c"
_FLAGS = {
    "parity": ["-O2", "-fno-fast-math", "-ffp-contract=off"],
    "timing": ["-O3", "-fno-fast-math", "-ffp-contract=off", "-fopenmp"],
}


def _lib_path(kind: str) -> Path:
    return _HERE / f"libbitlinear_oracle_{kind}.so"


def build_oracle(kind: str = "parity", force: bool = False) -> Path:
    """Compile the C oracle with gcc; returns the shared object's path."""
    out = _lib_path(kind)
    if not force and out.exists() and out.stat().st_mtime >= _SRC.stat().st_mtime:
        return out
    tmp = out.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", *_FLAGS[kind], "-std=gnu11", "-shared", "-fPIC", "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


_i64 = ctypes.c_int64
_p = ctypes.c_void_p


class Oracle:
    """Thin numpy wrapper; every method mirrors one C function."""

    def __init__(self, kind: str = "parity"):
        self.kind = kind
        self.lib = ctypes.CDLL(str(build_oracle(kind)))
        L = self.lib
        L.oracle_absmean.argtypes = [_p, _i64, _i64, _p]
        L.oracle_quantize_weights.argtypes = [_p, _i64, _i64, ctypes.c_float, _p, _p]
        L.oracle_packed_bytes.argtypes = [_i64, _i64]
        L.oracle_packed_bytes.restype = _i64
        L.oracle_pack_weights.argtypes = [_p, _i64, _i64, _p]
        L.oracle_unpack_weights.argtypes = [_p, _i64, _i64, _p]
        L.oracle_packed_bytes_trits.argtypes = [_i64, _i64]
        L.oracle_packed_bytes_trits.restype = _i64
        L.oracle_pack_weights_trits.argtypes = [_p, _i64, _i64, _p]
        L.oracle_unpack_weights_trits.argtypes = [_p, _i64, _i64, _p]
        L.oracle_quantize_acts.argtypes = [_p, _i64, _i64, _p, _p, _p]
        L.oracle_rmsnorm_quantize_acts.argtypes = [_p, _p, ctypes.c_float, _i64, _i64, _p, _p, _p, _p]
        L.oracle_rmsnorm_mean_square.argtypes = [_p, _i64, _i64, _p]
        L.oracle_swiglu_quantize_acts.argtypes = [_p, _p, _i64, _i64, _p, _p, _p, _p]
        L.oracle_quantize_acts_bits.argtypes = [_p, _i64, _i64, ctypes.c_int, _p, _p, _p]
        L.oracle_dequant_bits.argtypes = [_p, _p, ctypes.c_float, _i64, _i64, ctypes.c_int, _p]
        L.oracle_matmul_i32.argtypes = [_p, _p, _i64, _i64, _i64, _p]
        L.oracle_dequant.argtypes = [_p, _p, ctypes.c_float, _i64, _i64, _p]
        L.oracle_forward.argtypes = [_p, ctypes.c_float, _p, _i64, _i64, _i64, _p, _p, _p, _p, _p]
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_set_num_threads.argtypes = [ctypes.c_int]
        L.oracle_set_num_threads.restype = None

    @staticmethod
    def _c(a: np.ndarray, dtype) -> np.ndarray:
        a = np.ascontiguousarray(a, dtype=dtype)
        return a

    @staticmethod
    def _ptr(a: np.ndarray):
        return a.ctypes.data_as(_p)

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise ValueError(f"oracle {what} failed with code {rc}")

    def num_threads(self) -> int:
        return int(self.lib.oracle_num_threads())

    def set_num_threads(self, n: int) -> None:
        """Timing build only: threads used by the outer loops from now on (no effect on results)."""
        self.lib.oracle_set_num_threads(int(n))

    def absmean(self, W: np.ndarray) -> np.float32:
        W = self._c(W, np.float32)
        N, K = W.shape
        g = np.zeros(1, np.float32)
        self._check(self.lib.oracle_absmean(self._ptr(W), N, K, self._ptr(g)), "absmean")
        return g[0]

    def quantize_weights(self, W: np.ndarray, eps: float = 1e-5):
        """Eq. 1-3 -> (T int8 [N,K] in {-1,0,1}, gamma float32)."""
        W = self._c(W, np.float32)
        N, K = W.shape
        T = np.empty((N, K), np.int8)
        g = np.zeros(1, np.float32)
        rc = self.lib.oracle_quantize_weights(self._ptr(W), N, K, ctypes.c_float(eps), self._ptr(T), self._ptr(g))
        self._check(rc, "quantize_weights")
        return T, g[0]

    def packed_bytes(self, N: int, K: int) -> int:
        return int(self.lib.oracle_packed_bytes(N, K))

    def pack_weights(self, T: np.ndarray) -> np.ndarray:
        T = self._c(T, np.int8)
        N, K = T.shape
        nbytes = self.packed_bytes(N, K)
        if nbytes < 0:
            raise ValueError("N must be a positive multiple of 16")
        out = np.empty(nbytes, np.uint8)
        self._check(self.lib.oracle_pack_weights(self._ptr(T), N, K, self._ptr(out)), "pack_weights")
        return out

    def unpack_weights(self, packed: np.ndarray, N: int, K: int) -> np.ndarray:
        packed = self._c(packed, np.uint8)
        T = np.empty((N, K), np.int8)
        self._check(self.lib.oracle_unpack_weights(self._ptr(packed), N, K, self._ptr(T)), "unpack_weights")
        return T

    def packed_bytes_trits(self, N: int, K: int) -> int:
        return int(self.lib.oracle_packed_bytes_trits(N, K))

    def pack_weights_trits(self, T: np.ndarray) -> np.ndarray:
        """The base-3 storage: five weights per byte, tiles of 80 rows x 64 columns."""
        T = self._c(T, np.int8)
        N, K = T.shape
        nbytes = self.packed_bytes_trits(N, K)
        if nbytes < 0:
            raise ValueError("N must be a positive multiple of 16")
        out = np.empty(nbytes, np.uint8)
        self._check(self.lib.oracle_pack_weights_trits(self._ptr(T), N, K, self._ptr(out)), "pack_weights_trits")
        return out

    def unpack_weights_trits(self, packed: np.ndarray, N: int, K: int) -> np.ndarray:
        packed = self._c(packed, np.uint8)
        T = np.empty((N, K), np.int8)
        self._check(self.lib.oracle_unpack_weights_trits(self._ptr(packed), N, K, self._ptr(T)), "unpack_weights_trits")
        return T

    def quantize_acts(self, X_bf16_bits: np.ndarray):
        """-> (Xq int8 [M,K], beta float32 [M], rowsum int32 [M])."""
        X = self._c(X_bf16_bits, np.uint16)
        M, K = X.shape
        Xq = np.empty((M, K), np.int8)
        beta = np.empty(M, np.float32)
        rs = np.empty(M, np.int32)
        rc = self.lib.oracle_quantize_acts(self._ptr(X), M, K, self._ptr(Xq), self._ptr(beta), self._ptr(rs))
        self._check(rc, "quantize_acts")
        return Xq, beta, rs

    def quantize_acts_bits(self, X_bf16_bits: np.ndarray, bits: int):
        """The activation quantiser with Q_b = 2^(bits-1) - 1 -> (Xq int8 [M,K], beta float32 [M], rowsum int32 [M])."""
        X = self._c(X_bf16_bits, np.uint16)
        M, K = X.shape
        Xq = np.empty((M, K), np.int8)
        beta = np.empty(M, np.float32)
        rs = np.empty(M, np.int32)
        rc = self.lib.oracle_quantize_acts_bits(self._ptr(X), M, K, int(bits), self._ptr(Xq), self._ptr(beta), self._ptr(rs))
        self._check(rc, "quantize_acts_bits")
        return Xq, beta, rs

    def dequant_bits(self, acc: np.ndarray, beta: np.ndarray, gamma, bits: int) -> np.ndarray:
        acc = self._c(acc, np.int32)
        beta = self._c(beta, np.float32)
        M, N = acc.shape
        Y = np.empty((M, N), np.uint16)
        rc = self.lib.oracle_dequant_bits(self._ptr(acc), self._ptr(beta), ctypes.c_float(float(gamma)), M, N, int(bits),
                                          self._ptr(Y))
        self._check(rc, "dequant_bits")
        return Y

    def rmsnorm_quantize_acts(self, H_bf16_bits: np.ndarray, gain: np.ndarray, eps_n: float, return_x: bool = False):
        """RMSNorm (gain, eps_n) followed by the activation quantiser -> (Xq, beta, rowsum[, x float32 [M,K]])."""
        H = self._c(H_bf16_bits, np.uint16)
        g = self._c(gain, np.float32)
        M, K = H.shape
        assert g.shape == (K,)
        Xq = np.empty((M, K), np.int8)
        beta = np.empty(M, np.float32)
        rs = np.empty(M, np.int32)
        x = np.empty((M, K), np.float32) if return_x else None
        rc = self.lib.oracle_rmsnorm_quantize_acts(self._ptr(H), self._ptr(g), ctypes.c_float(float(eps_n)), M, K,
                                                   self._ptr(Xq), self._ptr(beta), self._ptr(rs),
                                                   self._ptr(x) if return_x else None)
        self._check(rc, "rmsnorm_quantize_acts")
        return (Xq, beta, rs, x) if return_x else (Xq, beta, rs)

    def rmsnorm_mean_square(self, H_bf16_bits: np.ndarray) -> np.ndarray:
        """The fp32 mean square of every token as the RMSNorm front forms it -> float32 [M]."""
        H = self._c(H_bf16_bits, np.uint16)
        M, K = H.shape
        mean = np.empty(M, np.float32)
        self._check(self.lib.oracle_rmsnorm_mean_square(self._ptr(H), M, K, self._ptr(mean)), "rmsnorm_mean_square")
        return mean

    def swiglu_quantize_acts(self, G_bf16_bits: np.ndarray, U_bf16_bits: np.ndarray, return_h: bool = False):
        """h = silu(g) * u in fp32 followed by the activation quantiser -> (Xq, beta, rowsum[, h float32 [M,K]])."""
        G = self._c(G_bf16_bits, np.uint16)
        U = self._c(U_bf16_bits, np.uint16)
        M, K = G.shape
        assert U.shape == (M, K)
        Xq = np.empty((M, K), np.int8)
        beta = np.empty(M, np.float32)
        rs = np.empty(M, np.int32)
        h = np.empty((M, K), np.float32) if return_h else None
        rc = self.lib.oracle_swiglu_quantize_acts(self._ptr(G), self._ptr(U), M, K, self._ptr(Xq), self._ptr(beta),
                                                  self._ptr(rs), self._ptr(h) if return_h else None)
        self._check(rc, "swiglu_quantize_acts")
        return (Xq, beta, rs, h) if return_h else (Xq, beta, rs)

    def matmul_i32(self, Xq: np.ndarray, T: np.ndarray) -> np.ndarray:
        Xq = self._c(Xq, np.int8)
        T = self._c(T, np.int8)
        M, K = Xq.shape
        N, K2 = T.shape
        assert K == K2
        acc = np.empty((M, N), np.int32)
        self._check(self.lib.oracle_matmul_i32(self._ptr(Xq), self._ptr(T), M, K, N, self._ptr(acc)), "matmul_i32")
        return acc

    def dequant(self, acc: np.ndarray, beta: np.ndarray, gamma) -> np.ndarray:
        acc = self._c(acc, np.int32)
        beta = self._c(beta, np.float32)
        M, N = acc.shape
        Y = np.empty((M, N), np.uint16)
        rc = self.lib.oracle_dequant(self._ptr(acc), self._ptr(beta), ctypes.c_float(float(gamma)), M, N, self._ptr(Y))
        self._check(rc, "dequant")
        return Y

    def forward(self, T: np.ndarray, gamma, X_bf16_bits: np.ndarray, return_all: bool = False):
        """Whole forward for ternary T [N,K]; returns bf16 bit patterns [M,N]."""
        T = self._c(T, np.int8)
        X = self._c(X_bf16_bits, np.uint16)
        N, K = T.shape
        M, K2 = X.shape
        assert K == K2
        Xq = np.empty((M, K), np.int8)
        beta = np.empty(M, np.float32)
        rs = np.empty(M, np.int32)
        acc = np.empty((M, N), np.int32)
        Y = np.empty((M, N), np.uint16)
        rc = self.lib.oracle_forward(self._ptr(T), ctypes.c_float(float(gamma)), self._ptr(X), M, K, N,
                                     self._ptr(Xq), self._ptr(beta), self._ptr(rs), self._ptr(acc), self._ptr(Y))
        self._check(rc, "forward")
        if return_all:
            return Y, acc, Xq, beta, rs
        return Y


_cache: dict[str, Oracle] = {}


def load_oracle(kind: str = "parity") -> Oracle:
    if kind not in _cache:
        _cache[kind] = Oracle(kind)
    return _cache[kind]


def bf16_bits_to_float32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a reinterpretation)."""
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)
