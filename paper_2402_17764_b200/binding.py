"""ctypes binding of libbitlinear_b200.so: argument marshalling only.

Function names match the C ABI (include/bitlinear.h).  Tensors are torch CUDA
tensors used purely as device memory; `stream` defaults to torch's current
stream.  There is no fallback: if the shared library is missing or a call
returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libbitlinear_b200.so"

OK = 0
ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT, ERR_RANGE, ERR_BADCODE = range(-1, -10, -1)
PATH_AUTO, PATH_DP4A, PATH_MMA, PATH_TCGEN05 = 0, 1, 2, 3

EXPORTS = [
    "bitlinear_status_string",
    "bitlinear_packed_bytes",
    "bitlinear_workspace_bytes",
    "bitlinear_quantize_weights",
    "bitlinear_quantize_acts",
    "bitlinear_rmsnorm_quantize_acts",
    "bitlinear_swiglu_quantize_acts",
    "bitlinear_quantize_acts_bits",
    "bitlinear_forward",
    "bitlinear_forward_act_bits",
    "bitlinear_forward_rmsnorm",
    "bitlinear_forward_swiglu",
    "bitlinear_forward_static",
    "bitlinear_sequence_workspace_bytes",
    "bitlinear_sequence_create",
    "bitlinear_sequence_create_rmsnorm",
    "bitlinear_sequence_create_swiglu",
    "bitlinear_forward_sequence",
    "bitlinear_forward_sequence_stage",
    "bitlinear_sequence_destroy",
    "bitlinear_matmul_i32",
    "bitlinear_unpack_weights",
    "bitlinear_validate_packed",
    "bitlinear_packed_bytes_trits",
    "bitlinear_quantize_weights_trits",
    "bitlinear_forward_trits",
    "bitlinear_sequence_create_trits",
    "bitlinear_matmul_i32_trits",
    "bitlinear_unpack_weights_trits",
    "bitlinear_probe_int8_peak",
    "bitlinear_test_expire_next_wait",
    "bitlinear_poll_status",
]


class BitLinearError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class LayerDesc(ctypes.Structure):
    _fields_ = [
        ("packed", ctypes.c_void_p),
        ("gamma", ctypes.c_void_p),
        ("X", ctypes.c_void_p),
        ("Y", ctypes.c_void_p),
        ("M", ctypes.c_int64),
        ("K", ctypes.c_int64),
        ("N", ctypes.c_int64),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2402_17764_b200.build` "
            "(the BitLinear path has no CPU or PyTorch fallback)")
    L = ctypes.CDLL(str(LIB_PATH))
    i64, vp, sz, ci, cf = ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_float
    L.bitlinear_status_string.argtypes = [ci]
    L.bitlinear_status_string.restype = ctypes.c_char_p
    L.bitlinear_packed_bytes.argtypes = [i64, i64]
    L.bitlinear_packed_bytes.restype = sz
    L.bitlinear_workspace_bytes.argtypes = [i64, i64, i64]
    L.bitlinear_workspace_bytes.restype = sz
    L.bitlinear_quantize_weights.argtypes = [vp, i64, i64, cf, vp, vp, vp]
    L.bitlinear_quantize_acts.argtypes = [vp, i64, i64, vp, vp, vp, vp]
    L.bitlinear_forward.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, sz, vp]
    L.bitlinear_rmsnorm_quantize_acts.argtypes = [vp, vp, cf, i64, i64, vp, vp, vp, vp]
    L.bitlinear_forward_rmsnorm.argtypes = [vp, vp, vp, vp, cf, i64, i64, i64, vp, vp, sz, vp]
    L.bitlinear_swiglu_quantize_acts.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    L.bitlinear_forward_swiglu.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, vp, sz, vp]
    L.bitlinear_quantize_acts_bits.argtypes = [vp, i64, i64, ci, vp, vp, vp, vp]
    L.bitlinear_forward_act_bits.argtypes = [vp, vp, vp, i64, i64, i64, ci, vp, vp, sz, vp]
    L.bitlinear_forward_static.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp]
    L.bitlinear_sequence_workspace_bytes.argtypes = [ctypes.POINTER(LayerDesc), ci]
    L.bitlinear_sequence_workspace_bytes.restype = sz
    L.bitlinear_sequence_create.argtypes = [ctypes.POINTER(LayerDesc), ci, vp, sz, ctypes.POINTER(vp)]
    L.bitlinear_sequence_create_rmsnorm.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(vp), cf, ci, vp, sz,
                                                    ctypes.POINTER(vp)]
    L.bitlinear_sequence_create_swiglu.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(vp), ctypes.POINTER(vp), cf,
                                                   ci, vp, sz, ctypes.POINTER(vp)]
    L.bitlinear_forward_sequence.argtypes = [vp, vp]
    L.bitlinear_forward_sequence_stage.argtypes = [vp, ci, vp]
    L.bitlinear_sequence_destroy.argtypes = [vp]
    L.bitlinear_sequence_destroy.restype = None
    L.bitlinear_matmul_i32.argtypes = [vp, vp, i64, i64, i64, vp, ci, vp, sz, vp]
    L.bitlinear_unpack_weights.argtypes = [vp, i64, i64, vp, vp]
    L.bitlinear_poll_status.argtypes = [vp, vp, ctypes.POINTER(ci)]
    L.bitlinear_validate_packed.argtypes = [vp, i64, i64, vp, vp]
    L.bitlinear_packed_bytes_trits.argtypes = [i64, i64]
    L.bitlinear_packed_bytes_trits.restype = sz
    L.bitlinear_quantize_weights_trits.argtypes = [vp, i64, i64, cf, vp, vp, vp]
    L.bitlinear_forward_trits.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, sz, vp]
    L.bitlinear_sequence_create_trits.argtypes = [ctypes.POINTER(LayerDesc), ci, vp, sz, ctypes.POINTER(vp)]
    L.bitlinear_matmul_i32_trits.argtypes = [vp, vp, i64, i64, i64, vp, vp, sz, vp]
    L.bitlinear_unpack_weights_trits.argtypes = [vp, i64, i64, vp, vp]
    L.bitlinear_probe_int8_peak.argtypes = [ci, vp, ctypes.POINTER(i64), vp]
    L.bitlinear_test_expire_next_wait.argtypes = [ctypes.c_uint32, ci]
    L.bitlinear_test_expire_next_wait.restype = None
    _lib = L
    return L


def status_string(status: int) -> str:
    return load_library().bitlinear_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise BitLinearError(status, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def packed_bytes(N: int, K: int) -> int:
    return int(load_library().bitlinear_packed_bytes(N, K))


def workspace_bytes(M: int, N: int, K: int) -> int:
    return int(load_library().bitlinear_workspace_bytes(M, N, K))


def alloc_workspace(M: int, N: int, K: int, device="cuda") -> torch.Tensor:
    n = workspace_bytes(M, N, K)
    if n == 0:
        raise BitLinearError(ERR_SHAPE, "bitlinear_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def quantize_weights(W: torch.Tensor, eps: float = 1e-5, packed: torch.Tensor | None = None,
                     gamma: torch.Tensor | None = None, stream=None):
    """bitlinear_quantize_weights: fp32 [N, K] -> (packed uint8 buffer, gamma fp32[1])."""
    N, K = W.shape
    if packed is None:
        packed = torch.empty(max(packed_bytes(N, K), 16), dtype=torch.uint8, device=W.device)
    if gamma is None:
        gamma = torch.empty(1, dtype=torch.float32, device=W.device)
    st = load_library().bitlinear_quantize_weights(_ptr(W), N, K, float(eps), _ptr(packed), _ptr(gamma), _stream(stream))
    _check(st, "bitlinear_quantize_weights")
    return packed, gamma


def packed_bytes_trits(N: int, K: int) -> int:
    return int(load_library().bitlinear_packed_bytes_trits(N, K))


def quantize_weights_trits(W: torch.Tensor, eps: float = 1e-5, packed: torch.Tensor | None = None,
                           gamma: torch.Tensor | None = None, stream=None):
    """bitlinear_quantize_weights_trits: fp32 [N, K] -> (base-3 packed uint8 buffer, gamma fp32[1])."""
    N, K = W.shape
    if packed is None:
        packed = torch.empty(packed_bytes_trits(N, K), dtype=torch.uint8, device=W.device)
    if gamma is None:
        gamma = torch.empty(1, dtype=torch.float32, device=W.device)
    st = load_library().bitlinear_quantize_weights_trits(_ptr(W), N, K, float(eps), _ptr(packed), _ptr(gamma), _stream(stream))
    _check(st, "bitlinear_quantize_weights_trits")
    return packed, gamma


def forward_trits(packed: torch.Tensor, gamma: torch.Tensor, X: torch.Tensor, N: int, Y: torch.Tensor | None = None,
                  workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_forward_trits: bf16 [M, K] (M <= 8) -> bf16 [M, N] on base-3 packed weights."""
    M, K = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, X.device)
    st = load_library().bitlinear_forward_trits(_ptr(packed), _ptr(gamma), _ptr(X), M, K, N, _ptr(Y), _ptr(workspace),
                                                workspace.numel(), _stream(stream))
    _check(st, "bitlinear_forward_trits")
    return Y


def matmul_i32_trits(packed: torch.Tensor, Xq: torch.Tensor, N: int, workspace: torch.Tensor | None = None,
                     stream=None) -> torch.Tensor:
    """bitlinear_matmul_i32_trits (test hook): int8 [M, K] x base-3 packed [N, K] -> int32 [M, N]."""
    M, K = Xq.shape
    acc = torch.empty((M, N), dtype=torch.int32, device=Xq.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, Xq.device)
    st = load_library().bitlinear_matmul_i32_trits(_ptr(packed), _ptr(Xq), M, K, N, _ptr(acc), _ptr(workspace),
                                                   workspace.numel(), _stream(stream))
    _check(st, "bitlinear_matmul_i32_trits")
    return acc


def unpack_weights_trits(packed: torch.Tensor, N: int, K: int, stream=None) -> torch.Tensor:
    """bitlinear_unpack_weights_trits (test hook): -> int8 [N, K] in {-1, 0, 1}."""
    T = torch.empty((N, K), dtype=torch.int8, device=packed.device)
    st = load_library().bitlinear_unpack_weights_trits(_ptr(packed), N, K, _ptr(T), _stream(stream))
    _check(st, "bitlinear_unpack_weights_trits")
    return T


def quantize_acts(X: torch.Tensor, stream=None):
    """bitlinear_quantize_acts: bf16 [M, K] -> (Xq int8 [M, K], beta fp32 [M], rowsum int32 [M])."""
    M, K = X.shape
    Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    beta = torch.empty(max(M, 1), dtype=torch.float32, device=X.device)[:M]
    rowsum = torch.empty(max(M, 1), dtype=torch.int32, device=X.device)[:M]
    st = load_library().bitlinear_quantize_acts(_ptr(X), M, K, _ptr(Xq), _ptr(beta), _ptr(rowsum), _stream(stream))
    _check(st, "bitlinear_quantize_acts")
    return Xq, beta, rowsum


def rmsnorm_quantize_acts(H: torch.Tensor, gain: torch.Tensor, norm_eps: float, stream=None):
    """bitlinear_rmsnorm_quantize_acts: bf16 [M, K], fp32 gain [K] -> (Xq int8 [M, K], beta fp32 [M], rowsum int32 [M])."""
    M, K = H.shape
    Xq = torch.empty((M, K), dtype=torch.int8, device=H.device)
    beta = torch.empty(max(M, 1), dtype=torch.float32, device=H.device)[:M]
    rowsum = torch.empty(max(M, 1), dtype=torch.int32, device=H.device)[:M]
    st = load_library().bitlinear_rmsnorm_quantize_acts(_ptr(H), _ptr(gain), float(norm_eps), M, K, _ptr(Xq), _ptr(beta),
                                                        _ptr(rowsum), _stream(stream))
    _check(st, "bitlinear_rmsnorm_quantize_acts")
    return Xq, beta, rowsum


def forward_rmsnorm(packed: torch.Tensor, gamma: torch.Tensor, H: torch.Tensor, gain: torch.Tensor, norm_eps: float, N: int,
                    Y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_forward_rmsnorm: BitLinear(RMSNorm(H)), bf16 [M, K] -> bf16 [M, N]."""
    M, K = H.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=H.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, H.device)
    st = load_library().bitlinear_forward_rmsnorm(_ptr(packed), _ptr(gamma), _ptr(H), _ptr(gain), float(norm_eps), M, K, N,
                                                  _ptr(Y), _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "bitlinear_forward_rmsnorm")
    return Y


def quantize_acts_bits(X: torch.Tensor, act_bits: int, stream=None):
    """bitlinear_quantize_acts_bits: bf16 [M, K] -> (Xq int8 [M, K] with |q| <= 2^(act_bits-1) - 1, beta, rowsum)."""
    M, K = X.shape
    Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    beta = torch.empty(max(M, 1), dtype=torch.float32, device=X.device)[:M]
    rowsum = torch.empty(max(M, 1), dtype=torch.int32, device=X.device)[:M]
    st = load_library().bitlinear_quantize_acts_bits(_ptr(X), M, K, int(act_bits), _ptr(Xq), _ptr(beta), _ptr(rowsum),
                                                     _stream(stream))
    _check(st, "bitlinear_quantize_acts_bits")
    return Xq, beta, rowsum


def forward_act_bits(packed: torch.Tensor, gamma: torch.Tensor, X: torch.Tensor, N: int, act_bits: int,
                     Y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_forward_act_bits: the forward with act_bits-bit activations, bf16 [M, K] -> bf16 [M, N]."""
    M, K = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, X.device)
    st = load_library().bitlinear_forward_act_bits(_ptr(packed), _ptr(gamma), _ptr(X), M, K, N, int(act_bits), _ptr(Y),
                                                   _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "bitlinear_forward_act_bits")
    return Y


def swiglu_quantize_acts(gate: torch.Tensor, up: torch.Tensor, stream=None):
    """bitlinear_swiglu_quantize_acts: bf16 gate, up [M, K] -> (Xq int8 [M, K], beta fp32 [M], rowsum int32 [M])."""
    M, K = gate.shape
    assert up.shape == gate.shape
    Xq = torch.empty((M, K), dtype=torch.int8, device=gate.device)
    beta = torch.empty(max(M, 1), dtype=torch.float32, device=gate.device)[:M]
    rowsum = torch.empty(max(M, 1), dtype=torch.int32, device=gate.device)[:M]
    st = load_library().bitlinear_swiglu_quantize_acts(_ptr(gate), _ptr(up), M, K, _ptr(Xq), _ptr(beta), _ptr(rowsum),
                                                       _stream(stream))
    _check(st, "bitlinear_swiglu_quantize_acts")
    return Xq, beta, rowsum


def forward_swiglu(packed: torch.Tensor, gamma: torch.Tensor, gate: torch.Tensor, up: torch.Tensor, N: int,
                   Y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_forward_swiglu: BitLinear(silu(gate) * up), bf16 [M, K] x 2 -> bf16 [M, N]."""
    M, K = gate.shape
    assert up.shape == gate.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=gate.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, gate.device)
    st = load_library().bitlinear_forward_swiglu(_ptr(packed), _ptr(gamma), _ptr(gate), _ptr(up), M, K, N, _ptr(Y),
                                                 _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "bitlinear_forward_swiglu")
    return Y


def forward(packed: torch.Tensor, gamma: torch.Tensor, X: torch.Tensor, N: int, Y: torch.Tensor | None = None,
            workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_forward: bf16 [M, K] -> bf16 [M, N]."""
    M, K = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, X.device)
    st = load_library().bitlinear_forward(_ptr(packed), _ptr(gamma), _ptr(X), M, K, N, _ptr(Y), _ptr(workspace),
                                          workspace.numel(), _stream(stream))
    _check(st, "bitlinear_forward")
    return Y


def forward_static(packed: torch.Tensor, gamma: torch.Tensor, X: torch.Tensor, N: int, Y: torch.Tensor,
                   stream=None) -> torch.Tensor:
    """bitlinear_forward_static: the forward on the library's own scratch; the caller supplies Y, nothing is allocated."""
    M, K = X.shape
    st = load_library().bitlinear_forward_static(_ptr(packed), _ptr(gamma), _ptr(X), M, K, N, _ptr(Y), _stream(stream))
    _check(st, "bitlinear_forward_static")
    return Y


def matmul_i32(packed: torch.Tensor, Xq: torch.Tensor, N: int, path: int = PATH_AUTO,
               workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """bitlinear_matmul_i32 (test hook): int8 [M, K] x packed [N, K] -> int32 [M, N]."""
    M, K = Xq.shape
    acc = torch.empty((M, N), dtype=torch.int32, device=Xq.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, Xq.device)
    st = load_library().bitlinear_matmul_i32(_ptr(packed), _ptr(Xq), M, K, N, _ptr(acc), int(path), _ptr(workspace),
                                             workspace.numel(), _stream(stream))
    _check(st, "bitlinear_matmul_i32")
    return acc


def unpack_weights(packed: torch.Tensor, N: int, K: int, stream=None) -> torch.Tensor:
    """bitlinear_unpack_weights (test hook): -> int8 [N, K] in {-1, 0, 1}."""
    T = torch.empty((N, K), dtype=torch.int8, device=packed.device)
    st = load_library().bitlinear_unpack_weights(_ptr(packed), N, K, _ptr(T), _stream(stream))
    _check(st, "bitlinear_unpack_weights")
    return T


def validate_packed(packed: torch.Tensor, N: int, K: int, stream=None) -> int:
    """bitlinear_validate_packed: -> number of 2-bit fields that hold the unused code 3 (0: the buffer is sound)."""
    bad = torch.empty(1, dtype=torch.int32, device=packed.device)
    st = load_library().bitlinear_validate_packed(_ptr(packed), N, K, _ptr(bad), _stream(stream))
    if st not in (OK, ERR_BADCODE):
        _check(st, "bitlinear_validate_packed")
    return int(bad.item())


def probe_int8_peak(iters: int, status: torch.Tensor, stream=None) -> int:
    """bitlinear_probe_int8_peak (measurement aid): enqueues the MMA issue loop; -> integer operations of the launch."""
    ops = ctypes.c_int64(0)
    st = load_library().bitlinear_probe_int8_peak(int(iters), _ptr(status), ctypes.byref(ops), _stream(stream))
    _check(st, "bitlinear_probe_int8_peak")
    return int(ops.value)


def test_expire_next_wait(limit_us: int, skip_arrive: bool):
    """bitlinear_test_expire_next_wait (test hook): arms the next matmul launch; see include/bitlinear.h."""
    load_library().bitlinear_test_expire_next_wait(int(limit_us), 1 if skip_arrive else 0)


def poll_status(workspace: torch.Tensor, stream=None) -> int:
    out = ctypes.c_int(0)
    st = load_library().bitlinear_poll_status(_ptr(workspace), _stream(stream), ctypes.byref(out))
    _check(st, "bitlinear_poll_status")
    return int(out.value)


class Sequence:
    """bitlinear_sequence_*: a fixed list of independent BitLinear forwards run by one persistent launch.

    `layers` is a list of (packed, gamma, X, Y, N) with torch tensors; the object keeps them alive.
    `gains` (optional): one fp32 gain vector [K] or None per layer; those layers get an RMSNorm with `norm_eps` in front
    of their activation quantiser (bitlinear_sequence_create_rmsnorm).
    `ups` (optional): one bf16 tensor [M, K] or None per layer; those layers quantise silu(X) * up
    (bitlinear_sequence_create_swiglu).
    `trits`: the packed weights are in the base-3 format (bitlinear_sequence_create_trits).
    """

    def __init__(self, layers, device="cuda", gains=None, norm_eps: float = 1e-5, ups=None, trits: bool = False):
        L = load_library()
        self._keep = list(layers)
        self._gains = list(gains) if gains is not None else None
        self._ups = list(ups) if ups is not None else None
        n = len(self._keep)
        arr = (LayerDesc * n)()
        for i, (packed, gamma, X, Y, N) in enumerate(self._keep):
            M, K = X.shape
            arr[i] = LayerDesc(_ptr(packed), _ptr(gamma), _ptr(X), _ptr(Y), M, K, N)
        nbytes = int(L.bitlinear_sequence_workspace_bytes(arr, n))
        if nbytes == 0:
            raise BitLinearError(ERR_SHAPE, "bitlinear_sequence_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        handle = ctypes.c_void_p()
        def pointers(tensors):
            assert len(tensors) == n
            return (ctypes.c_void_p * n)(*[(_ptr(x) if x is not None else None) for x in tensors])

        if trits:
            assert self._ups is None and self._gains is None
            st = L.bitlinear_sequence_create_trits(arr, n, _ptr(self.workspace), nbytes, ctypes.byref(handle))
        elif self._ups is not None:
            st = L.bitlinear_sequence_create_swiglu(arr, pointers(self._gains) if self._gains is not None else None,
                                                    pointers(self._ups), float(norm_eps), n, _ptr(self.workspace), nbytes,
                                                    ctypes.byref(handle))
        elif self._gains is None:
            st = L.bitlinear_sequence_create(arr, n, _ptr(self.workspace), nbytes, ctypes.byref(handle))
        else:
            assert len(self._gains) == n
            garr = (ctypes.c_void_p * n)(*[(_ptr(g) if g is not None else None) for g in self._gains])
            st = L.bitlinear_sequence_create_rmsnorm(arr, garr, float(norm_eps), n, _ptr(self.workspace), nbytes,
                                                     ctypes.byref(handle))
        _check(st, "bitlinear_sequence_create")
        self._handle = handle
        self.n = n

    def forward(self, stream=None):
        st = load_library().bitlinear_forward_sequence(self._handle, _stream(stream))
        _check(st, "bitlinear_forward_sequence")

    def forward_stage(self, stage: int, stream=None):
        """stage 1: activation quantiser; stage 2: matmul + dequantisation; 0: both."""
        st = load_library().bitlinear_forward_sequence_stage(self._handle, int(stage), _stream(stream))
        _check(st, "bitlinear_forward_sequence_stage")

    def close(self):
        if getattr(self, "_handle", None):
            load_library().bitlinear_sequence_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
