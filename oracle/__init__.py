"""CPU oracle for block-quantised matrix products: ctypes binding of qmm_oracle.c.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this
package; it exists so that the tests, the smoke check and the CPU-baseline leg
of the benchmark can compare the CUDA library against a plain definition.

The arithmetic lives in ``qmm_oracle.c`` (see ``qmm_oracle.h`` for what each
function computes and which conventions it follows).  This module only
marshals numpy arrays and builds the shared object with gcc on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

Q4 = 4
Q5 = 5
Q6 = 6
Q8 = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qmm_oracle.c")
_HDR = os.path.join(_HERE, "qmm_oracle.h")
_LIB = os.path.join(_HERE, "libqmm_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile qmm_oracle.c into libqmm_oracle.so beside it (gcc, OpenMP)."""
    stale = (
        force
        or not os.path.exists(_LIB)
        or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    )
    if stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
            lib.orc_h2f.restype = ctypes.c_float
            lib.orc_h2f.argtypes = [ctypes.c_uint16]
            lib.orc_f2h.restype = ctypes.c_uint16
            lib.orc_f2h.argtypes = [ctypes.c_float]
            lib.orc_block_bytes.restype = ctypes.c_size_t
            lib.orc_block_bytes.argtypes = [ci]
            lib.orc_canonical_bytes.restype = ctypes.c_size_t
            lib.orc_canonical_bytes.argtypes = [ci, i64, i64]
            lib.orc_quantize.argtypes = [ci, vp, i64, i64, vp]
            lib.orc_dequant.argtypes = [ci, vp, i64, i64, vp]
            lib.orc_gemm.argtypes = [ci, vp, i64, i64, vp, i64, i64, vp, vp]
            lib.orc_gemv.argtypes = [ci, vp, i64, i64, vp, vp, vp]
            lib.orc_gemm_f64.argtypes = [ci, vp, i64, i64, vp, i64, i64, vp, vp]
            lib.orc_route.argtypes = [vp, i64, i64, i64, vp, vp]
            lib.orc_permute.argtypes = [vp, i64, i64, i64, vp, vp]
            lib.orc_silu.restype = ctypes.c_double
            lib.orc_silu.argtypes = [ctypes.c_double]
            lib.orc_moe_tokens.argtypes = [ci, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, vp, i64, vp]
            lib.orc_num_threads.restype = ci
            _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError("oracle %s rejected its input (rc=%d)" % (what, rc))


def num_threads() -> int:
    return int(_load().orc_num_threads())


def h2f(h: int) -> float:
    return float(_load().orc_h2f(int(h) & 0xFFFF))


def f2h(f: float) -> int:
    return int(_load().orc_f2h(float(np.float32(f))))


def block_bytes(fmt: int) -> int:
    return int(_load().orc_block_bytes(fmt))


def canonical_bytes(fmt: int, N: int, K: int) -> int:
    return int(_load().orc_canonical_bytes(fmt, N, K))


def quantize(fmt: int, w: np.ndarray) -> np.ndarray:
    """fp32 W[N,K] -> canonical blocks (uint8, N*(K/32)*block_bytes)."""
    w = _c(w, np.float32)
    N, K = w.shape
    out = np.empty(canonical_bytes(fmt, N, K), dtype=np.uint8)
    _check(_load().orc_quantize(fmt, _ptr(w), N, K, _ptr(out)), "quantize")
    return out


def dequant(fmt: int, blocks: np.ndarray, N: int, K: int) -> np.ndarray:
    blocks = _c(blocks, np.uint8)
    assert blocks.size == canonical_bytes(fmt, N, K)
    w = np.empty((N, K), dtype=np.float32)
    _check(_load().orc_dequant(fmt, _ptr(blocks), N, K, _ptr(w)), "dequant")
    return w


def gemm(fmt: int, blocks: np.ndarray, N: int, K: int, X: np.ndarray):
    """X: fp16 [M,K] (np.float16 or uint16 bits).  Returns (Y, B) as float64 [M,N]."""
    blocks = _c(blocks, np.uint8)
    assert blocks.size == canonical_bytes(fmt, N, K)
    Xb = _c(X.view(np.uint16) if X.dtype == np.float16 else X, np.uint16)
    Xb = Xb.reshape(-1, K)
    M = Xb.shape[0]
    Y = np.empty((M, N), dtype=np.float64)
    B = np.empty((M, N), dtype=np.float64)
    _check(_load().orc_gemm(fmt, _ptr(blocks), N, K, _ptr(Xb), K, M, _ptr(Y), _ptr(B)), "gemm")
    return Y, B


def gemv(fmt: int, blocks: np.ndarray, N: int, K: int, x: np.ndarray):
    """x: fp16 [K].  Returns (y, B) as float64 [N]."""
    Y, B = gemm(fmt, blocks, N, K, x.reshape(1, K))
    return Y[0], B[0]


def gemm_f64(fmt: int, blocks: np.ndarray, N: int, K: int, X: np.ndarray):
    blocks = _c(blocks, np.uint8)
    assert blocks.size == canonical_bytes(fmt, N, K)
    Xd = _c(X, np.float64).reshape(-1, K)
    M = Xd.shape[0]
    Y = np.empty((M, N), dtype=np.float64)
    B = np.empty((M, N), dtype=np.float64)
    _check(_load().orc_gemm_f64(fmt, _ptr(blocks), N, K, _ptr(Xd), K, M, _ptr(Y), _ptr(B)), "gemm_f64")
    return Y, B


def route(logits: np.ndarray, topk: int):
    """logits fp32 [T,E] -> (idx int32 [T,topk], p float64 [T,topk])."""
    logits = _c(logits, np.float32)
    T, E = logits.shape
    idx = np.empty((T, topk), dtype=np.int32)
    p = np.empty((T, topk), dtype=np.float64)
    _check(_load().orc_route(_ptr(logits), T, E, topk, _ptr(idx), _ptr(p)), "route")
    return idx, p


def permute(idx: np.ndarray, E: int):
    """idx int32 [T,topk] -> (perm int32 [T*topk], offsets int32 [E+1])."""
    idx = _c(idx, np.int32)
    T, topk = idx.shape
    perm = np.empty(T * topk, dtype=np.int32)
    offs = np.empty(E + 1, dtype=np.int32)
    _check(_load().orc_permute(_ptr(idx), T, topk, E, _ptr(perm), _ptr(offs)), "permute")
    return perm, offs


def silu(g):
    g = np.asarray(g, dtype=np.float64)
    f = _load().orc_silu
    return np.vectorize(lambda v: f(float(v)), otypes=[np.float64])(g)


def moe_tokens(fmt, logits, X, w_gate, w_up, w_down, H, I, E, topk, tokens):
    """All-fp64 layer output for the listed tokens: float64 [len(tokens), H]."""
    logits = _c(logits, np.float32)
    T = logits.shape[0]
    Xb = _c(X.view(np.uint16) if X.dtype == np.float16 else X, np.uint16).reshape(T, H)
    wg, wu, wd = _c(w_gate, np.uint8), _c(w_up, np.uint8), _c(w_down, np.uint8)
    assert wg.size == E * canonical_bytes(fmt, I, H) and wu.size == wg.size
    assert wd.size == E * canonical_bytes(fmt, H, I)
    tok = _c(tokens, np.int32)
    out = np.empty((tok.size, H), dtype=np.float64)
    _check(_load().orc_moe_tokens(fmt, _ptr(logits), _ptr(Xb), _ptr(wg), _ptr(wu), _ptr(wd),
                                  T, H, I, E, topk, _ptr(tok), tok.size, _ptr(out)), "moe_tokens")
    return out
