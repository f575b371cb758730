"""Thin ctypes binding of libqmm.so (the C ABI declared in include/qmm.h).

Argument marshalling only: every step of every product runs in the CUDA
kernels of the library.  PyTorch is used for device memory and streams.  There
is no CPU fallback: if the shared library cannot be loaded, or a call fails,
an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
import threading

import torch

Q4 = 4
Q5 = 5
Q6 = 6
Q8 = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqmm.so")
_lock = threading.Lock()
_lib = None

STATUS_NAMES = {
    0: "QMM_OK", 1: "QMM_ERR_INVALID_ARG", 2: "QMM_ERR_SHAPE", 3: "QMM_ERR_ALIGNMENT",
    4: "QMM_ERR_WORKSPACE", 5: "QMM_ERR_UNSUPPORTED", 6: "QMM_ERR_CUDA", 7: "QMM_ERR_DEVICE_TIMEOUT",
    8: "QMM_ERR_BAD_WEIGHTS",
}

# every symbol include/qmm.h declares
EXPORTS = (
    "qmm_last_error", "qmm_version", "qmm_canonical_bytes", "qmm_packed_bytes", "qmm_pack",
    "qmm_dequant", "qmm_gemv_workspace_bytes", "qmm_gemv", "qmm_gemm_workspace_bytes", "qmm_gemm",
    "qmm_moe_workspace_bytes", "qmm_moe", "qmm_moe_route", "qmm_status_check", "qmm_gemv_static", "qmm_gemv_batch", "qmm_gemm_batch",
    "qmm_gemv_gate_up", "qmm_packed_check", "qmm_debug_config", "qmm_debug_wait_give_up",
    "qmm_chain_plan_bytes", "qmm_chain_workspace_bytes", "qmm_chain_build", "qmm_chain_run",
)


class QmmError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status
        self.message = message


class GemvProblem(ctypes.Structure):
    _fields_ = [("packed", ctypes.c_void_p), ("x_fp16", ctypes.c_void_p), ("y_fp16", ctypes.c_void_p),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64)]


class GemmProblem(ctypes.Structure):
    _fields_ = [("packed", ctypes.c_void_p), ("X_fp16", ctypes.c_void_p), ("Y_fp16", ctypes.c_void_p),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64), ("ldx", ctypes.c_int64), ("ldy", ctypes.c_int64)]


class ChainStage(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("x_stage", ctypes.c_int32), ("x_offset", ctypes.c_int64),
                ("x_fp16", ctypes.c_void_p), ("packed", ctypes.c_void_p), ("packed_up", ctypes.c_void_p),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64), ("y_fp16", ctypes.c_void_p)]


class ChainInfo(ctypes.Structure):
    _fields_ = [("magic", ctypes.c_int32), ("fmt", ctypes.c_int32), ("stages", ctypes.c_int32), ("grid", ctypes.c_int32),
                ("threads", ctypes.c_int32), ("smem_bytes", ctypes.c_int32), ("plan_bytes", ctypes.c_uint64),
                ("ws_bytes", ctypes.c_uint64), ("plan", ctypes.c_void_p), ("ws", ctypes.c_void_p)]


CHAIN_LINEAR = 0
CHAIN_GATE_UP_SILU = 1


class MoeArgs(ctypes.Structure):
    _fields_ = [
        ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("E", ctypes.c_int32),
        ("topk", ctypes.c_int32), ("fmt", ctypes.c_int32),
        ("logits", ctypes.c_void_p), ("X", ctypes.c_void_p),
        ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p),
        ("out", ctypes.c_void_p),
        ("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p),
        ("perm", ctypes.c_void_p), ("expert_offsets", ctypes.c_void_p),
        ("dbg_H", ctypes.c_void_p), ("dbg_D", ctypes.c_void_p),
        ("w_router", ctypes.c_void_p), ("router_logits", ctypes.c_void_p),
    ]


def lib() -> ctypes.CDLL:
    """Load libqmm.so (building it with nvcc first if it is not there)."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                from . import _build
                _build.build()
            L = ctypes.CDLL(LIB_PATH)
            i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
            L.qmm_last_error.restype = ctypes.c_char_p
            L.qmm_last_error.argtypes = []
            L.qmm_version.restype = ci
            L.qmm_canonical_bytes.restype = sz
            L.qmm_canonical_bytes.argtypes = [ci, i64, i64]
            L.qmm_packed_bytes.restype = sz
            L.qmm_packed_bytes.argtypes = [ci, i64, i64]
            L.qmm_pack.argtypes = [ci, vp, i64, i64, vp, vp]
            L.qmm_dequant.argtypes = [ci, vp, i64, i64, vp, vp]
            L.qmm_gemv_workspace_bytes.restype = sz
            L.qmm_gemv_workspace_bytes.argtypes = [ci, i64, i64]
            L.qmm_gemv.argtypes = [ci, vp, i64, i64, vp, vp, vp, sz, vp]
            L.qmm_gemv_static.argtypes = [ci, vp, i64, i64, vp, vp, vp]
            L.qmm_gemv_gate_up.argtypes = [ci, vp, vp, i64, i64, vp, vp, vp]
            L.qmm_gemv_batch.argtypes = [ci, ctypes.POINTER(GemvProblem), ci, vp]
            L.qmm_gemm_batch.argtypes = [ci, ctypes.POINTER(GemmProblem), ci, i64, vp]
            L.qmm_gemm_workspace_bytes.restype = sz
            L.qmm_gemm_workspace_bytes.argtypes = [ci, i64, i64, i64]
            L.qmm_gemm.argtypes = [ci, vp, i64, i64, vp, i64, vp, i64, i64, vp, sz, vp]
            L.qmm_moe_workspace_bytes.restype = sz
            L.qmm_moe_workspace_bytes.argtypes = [ctypes.POINTER(MoeArgs)]
            L.qmm_moe.argtypes = [ctypes.POINTER(MoeArgs), vp, sz, vp]
            L.qmm_moe_route.argtypes = [ctypes.POINTER(MoeArgs), vp, sz, vp]
            L.qmm_status_check.argtypes = [vp, vp]
            L.qmm_chain_plan_bytes.restype = sz
            L.qmm_chain_plan_bytes.argtypes = [ci, ctypes.POINTER(ChainStage), ci]
            L.qmm_chain_workspace_bytes.restype = sz
            L.qmm_chain_workspace_bytes.argtypes = [ci, ctypes.POINTER(ChainStage), ci]
            L.qmm_chain_build.argtypes = [ci, ctypes.POINTER(ChainStage), ci, vp, sz, vp, sz, ctypes.POINTER(ChainInfo), vp]
            L.qmm_chain_run.argtypes = [ctypes.POINTER(ChainInfo), vp]
            L.qmm_packed_check.argtypes = [ci, vp, i64, i64, vp, vp]
            L.qmm_debug_config.argtypes = [ctypes.c_char_p, ctypes.c_char_p]
            L.qmm_debug_wait_give_up.argtypes = [vp, i64, vp]
            _lib = L
    return _lib


def last_error() -> str:
    return lib().qmm_last_error().decode("utf-8", "replace")


def _check(status: int):
    if status != 0:
        raise QmmError(status, last_error())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dp(t):
    return 0 if t is None else t.data_ptr()


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def version() -> int:
    return lib().qmm_version()


def canonical_bytes(fmt: int, N: int, K: int) -> int:
    return lib().qmm_canonical_bytes(fmt, N, K)


def packed_bytes(fmt: int, N: int, K: int) -> int:
    n = lib().qmm_packed_bytes(fmt, N, K)
    if n == 0:
        raise QmmError(5, last_error())
    return n


def pack(fmt: int, canonical: torch.Tensor, N: int, K: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """canonical: uint8 CUDA tensor of canonical_bytes(fmt,N,K) bytes -> packed uint8 tensor."""
    assert canonical.is_cuda and canonical.dtype == torch.uint8 and canonical.is_contiguous()
    assert canonical.numel() == canonical_bytes(fmt, N, K)
    if out is None:
        out = torch.empty(packed_bytes(fmt, N, K), dtype=torch.uint8, device=canonical.device)
    _check(lib().qmm_pack(fmt, canonical.data_ptr(), N, K, out.data_ptr(), _stream()))
    return out


def dequant(fmt: int, packed: torch.Tensor, N: int, K: int) -> torch.Tensor:
    out = torch.empty((N, K), dtype=torch.float32, device=packed.device)
    _check(lib().qmm_dequant(fmt, packed.data_ptr(), N, K, out.data_ptr(), _stream()))
    return out


def gemv_workspace_bytes(fmt: int, N: int, K: int) -> int:
    return lib().qmm_gemv_workspace_bytes(fmt, N, K)


def gemv(fmt: int, packed: torch.Tensor, N: int, K: int, x: torch.Tensor,
         y: torch.Tensor | None = None, ws: torch.Tensor | None = None) -> torch.Tensor:
    """y = W x.  x: fp16 [K] CUDA tensor; returns fp16 [N]."""
    assert x.is_cuda and x.dtype == torch.float16 and x.numel() == K and x.is_contiguous()
    if y is None:
        y = torch.empty(N, dtype=torch.float16, device=x.device)
    if ws is None:
        need = gemv_workspace_bytes(fmt, N, K)
        ws = torch.empty(need, dtype=torch.uint8, device=x.device) if need else None
    _check(lib().qmm_gemv(fmt, packed.data_ptr(), N, K, x.data_ptr(), y.data_ptr(), _dp(ws), _nbytes(ws), _stream()))
    return y


def gemv_batch_problems(problems):
    """problems: iterable of (packed, N, K, x, y) tensors -> ctypes array for gemv_batch (keeps the tensors alive)."""
    problems = list(problems)
    arr = (GemvProblem * len(problems))()
    for i, (packed, N, K, x, y) in enumerate(problems):
        assert x.dtype == torch.float16 and x.numel() == K and y.dtype == torch.float16 and y.numel() == N
        arr[i] = GemvProblem(packed.data_ptr(), x.data_ptr(), y.data_ptr(), N, K)
    arr._keep = problems
    return arr


def gemv_batch(fmt: int, problems) -> None:
    """All products y_i = W_i x_i of the list in one launch.  `problems` is the array made by
    gemv_batch_problems (build it once and reuse it: the call only reads it)."""
    _check(lib().qmm_gemv_batch(fmt, problems, len(problems), _stream()))


def gemm_batch_problems(problems):
    """problems: iterable of (packed, N, K, X [M, K], Y [M, N]) tensors -> ctypes array for gemm_batch (keeps
    the tensors alive).  Row strides may exceed K / N; every X and Y has the same number of rows."""
    problems = list(problems)
    arr = (GemmProblem * len(problems))()
    for i, (packed, N, K, X, Y) in enumerate(problems):
        assert X.dtype == torch.float16 and X.dim() == 2 and X.shape[1] == K and X.stride(1) == 1
        assert Y.dtype == torch.float16 and Y.dim() == 2 and Y.shape == (X.shape[0], N) and Y.stride(1) == 1
        M = X.shape[0]
        arr[i] = GemmProblem(packed.data_ptr(), X.data_ptr(), Y.data_ptr(), N, K,
                             X.stride(0) if M > 1 else max(K, X.stride(0)), Y.stride(0) if M > 1 else max(N, Y.stride(0)))
    arr._keep = problems
    arr._M = problems[0][3].shape[0] if problems else 0
    return arr


def gemm_batch(fmt: int, problems) -> None:
    """All products Y_i = X_i W_i^T (M <= 8 rows each) of the list in one launch.  `problems` is the array
    made by gemm_batch_problems (build it once and reuse it: the call only reads it)."""
    _check(lib().qmm_gemm_batch(fmt, problems, len(problems), problems._M, _stream()))


GEMV_STATIC_SCRATCH_BYTES = 1 << 20


def gemv_gate_up(fmt: int, packed_gate: torch.Tensor, packed_up: torch.Tensor, N: int, K: int, x: torch.Tensor,
                 h: torch.Tensor | None = None) -> torch.Tensor:
    """h = fp16(silu(W_gate x) * (W_up x)) in one launch (both products kept in fp32 until the end)."""
    assert x.is_cuda and x.dtype == torch.float16 and x.numel() == K and x.is_contiguous()
    if h is None:
        h = torch.empty(N, dtype=torch.float16, device=x.device)
    assert h.is_cuda and h.dtype == torch.float16 and h.numel() == N and h.is_contiguous()
    _check(lib().qmm_gemv_gate_up(fmt, packed_gate.data_ptr(), packed_up.data_ptr(), N, K, x.data_ptr(), h.data_ptr(), _stream()))
    return h


def gemv_static(fmt: int, packed: torch.Tensor, N: int, K: int, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """y = W x through qmm_gemv_static: no workspace argument and no allocation anywhere.

    For callers that may not allocate device memory when they need the product (memory
    budget already handed out, allocator calls forbidden after start-up, no tolerance for
    the device-wide synchronisation an allocation implies).  The split-K scratch is a fixed
    array inside the library (GEMV_STATIC_SCRATCH_BYTES per GPU); shapes that need more
    raise QmmError (QMM_ERR_WORKSPACE).  `y` must be provided by the caller.  All calls on a
    device share that scratch: keep them on one stream.  Make the first call on each device
    outside any stream capture.
    """
    assert x.is_cuda and x.dtype == torch.float16 and x.numel() == K and x.is_contiguous()
    assert y.is_cuda and y.dtype == torch.float16 and y.numel() == N and y.is_contiguous()
    _check(lib().qmm_gemv_static(fmt, packed.data_ptr(), N, K, x.data_ptr(), y.data_ptr(), _stream()))
    return y


def gemm_workspace_bytes(fmt: int, M: int, N: int, K: int) -> int:
    return lib().qmm_gemm_workspace_bytes(fmt, M, N, K)


def gemm(fmt: int, packed: torch.Tensor, N: int, K: int, X: torch.Tensor,
         Y: torch.Tensor | None = None, ws: torch.Tensor | None = None) -> torch.Tensor:
    """Y = X W^T.  X: fp16 [M,K] (row stride >= K); returns fp16 [M,N]."""
    assert X.is_cuda and X.dtype == torch.float16 and X.dim() == 2 and X.shape[1] == K and X.stride(1) == 1
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
    assert Y.stride(1) == 1
    if ws is None:
        ws = torch.zeros(max(gemm_workspace_bytes(fmt, M, N, K), 256), dtype=torch.uint8, device=X.device)
    _check(lib().qmm_gemm(fmt, packed.data_ptr(), N, K, X.data_ptr(), X.stride(0) if M > 1 else max(K, X.stride(0)),
                          Y.data_ptr(), Y.stride(0) if M > 1 else max(N, Y.stride(0)), M,
                          ws.data_ptr(), _nbytes(ws), _stream()))
    return Y


def moe_args(fmt, T, H, I, E, topk, logits, X, w_gate, w_up, w_down, out,
             topk_idx=None, topk_w=None, perm=None, expert_offsets=None, dbg_H=None, dbg_D=None,
             w_router=None, router_logits=None) -> MoeArgs:
    a = MoeArgs(T, H, I, E, topk, fmt, _dp(logits), _dp(X), _dp(w_gate), _dp(w_up), _dp(w_down), _dp(out),
                _dp(topk_idx), _dp(topk_w), _dp(perm), _dp(expert_offsets), _dp(dbg_H), _dp(dbg_D),
                _dp(w_router), _dp(router_logits))
    # the struct holds raw device pointers only: keep the tensors alive as long as the struct
    a._keep = (logits, X, w_gate, w_up, w_down, out, topk_idx, topk_w, perm, expert_offsets, dbg_H, dbg_D, w_router, router_logits)
    return a


def moe_workspace_bytes(args: MoeArgs) -> int:
    n = lib().qmm_moe_workspace_bytes(ctypes.byref(args))
    if n == 0:
        raise QmmError(5, last_error())
    return n


def moe(args: MoeArgs, ws: torch.Tensor) -> None:
    _check(lib().qmm_moe(ctypes.byref(args), ws.data_ptr(), _nbytes(ws), _stream()))


def moe_route(args: MoeArgs, ws: torch.Tensor) -> None:
    _check(lib().qmm_moe_route(ctypes.byref(args), ws.data_ptr(), _nbytes(ws), _stream()))


def status_check(ws: torch.Tensor) -> None:
    _check(lib().qmm_status_check(ws.data_ptr(), _stream()))


class Chain:
    """A planned list of decode products (qmm_chain_build); run() is the one-launch hot-path call.

    stages: list of dicts with keys op, packed, N, K and either x (fp16 CUDA tensor) or x_stage (+ x_offset);
    optional packed_up (gate/up stages) and y (fp16 CUDA tensor receiving a plain copy of the output).
    The object keeps every tensor it refers to alive; the plan and workspace tensors are attributes."""

    def __init__(self, fmt: int, stages):
        self.fmt = fmt
        self._keep = []
        arr = (ChainStage * len(stages))()
        for i, s in enumerate(stages):
            x, y, up = s.get("x"), s.get("y"), s.get("packed_up")
            if x is not None:
                assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.numel() == s["K"]
            if y is not None:
                assert y.is_cuda and y.dtype == torch.float16 and y.is_contiguous() and y.numel() == s["N"]
            arr[i] = ChainStage(s.get("op", CHAIN_LINEAR), -1 if x is not None else s["x_stage"], s.get("x_offset", 0),
                                _dp(x), s["packed"].data_ptr(), _dp(up), s["N"], s["K"], _dp(y))
            self._keep.append((x, y, up, s["packed"]))
        self.stages = arr
        L = lib()
        plan_bytes = L.qmm_chain_plan_bytes(fmt, arr, len(arr))
        ws_bytes = L.qmm_chain_workspace_bytes(fmt, arr, len(arr))
        if plan_bytes == 0 or ws_bytes == 0:
            raise QmmError(1, last_error())
        self.plan = torch.empty(plan_bytes, dtype=torch.uint8, device="cuda")
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        self.info = ChainInfo()
        _check(L.qmm_chain_build(fmt, arr, len(arr), self.plan.data_ptr(), plan_bytes, self.ws.data_ptr(), ws_bytes,
                                 ctypes.byref(self.info), _stream()))

    def run(self) -> None:
        _check(lib().qmm_chain_run(ctypes.byref(self.info), _stream()))


def packed_check(fmt: int, packed: torch.Tensor, N: int, K: int, ws: torch.Tensor) -> None:
    """Enqueue the plausibility check of a packed buffer; status_check(ws) reports the outcome."""
    _check(lib().qmm_packed_check(fmt, packed.data_ptr(), N, K, ws.data_ptr(), _stream()))


def debug_config(name: str | None, value: str | None = None) -> None:
    """Set (or with value None clear) a debug knob; name None resets all of them."""
    enc = lambda v: None if v is None else str(v).encode()
    _check(lib().qmm_debug_config(enc(name), enc(value)))


def debug_wait_give_up(ws: torch.Tensor, limit_cycles: int) -> None:
    _check(lib().qmm_debug_wait_give_up(ws.data_ptr(), int(limit_cycles), _stream()))
