"""ctypes front end of the fp64 CPU attention oracle (``ave_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
CPU-baseline / reference legs of the benchmark.  The CUDA library and its
Python binding never import this package, and this package never imports them.

The functions take CPU ``torch.bfloat16`` tensors (or ``numpy.uint16`` arrays of
bf16 bit patterns) in the layouts documented in ``ave_oracle.h`` and return
``numpy.float64`` arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ave_oracle.c")
_HDR = os.path.join(_HERE, "ave_oracle.h")
_LIB = os.path.join(_HERE, "libave_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``ave_oracle.c`` with gcc into ``libave_oracle.so`` beside it."""
    newest_src = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest_src:
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            u16p = ctypes.POINTER(ctypes.c_uint16)
            f64p = ctypes.POINTER(ctypes.c_double)
            i64p = ctypes.POINTER(ctypes.c_int64)
            dims = [ctypes.c_int] * 6 + [ctypes.c_int, ctypes.c_float]
            lib.ave_oracle_attn_fwd.argtypes = [u16p, u16p, u16p, f64p, f64p, f64p] + dims
            lib.ave_oracle_attn_fwd.restype = ctypes.c_int
            lib.ave_oracle_attn_rows.argtypes = [u16p, u16p, u16p, i64p, ctypes.c_int64, f64p, f64p] + dims
            lib.ave_oracle_attn_rows.restype = ctypes.c_int
            lib.ave_oracle_bruteforce.argtypes = [u16p, u16p, u16p, f64p, f64p] + dims
            lib.ave_oracle_bruteforce.restype = ctypes.c_int
            lib.ave_oracle_gemm_tn.argtypes = [u16p, u16p, f64p] + [ctypes.c_int] * 3
            lib.ave_oracle_gemm_tn.restype = ctypes.c_int
            lib.ave_oracle_gemm_tn_entries.argtypes = [u16p, u16p, i64p, ctypes.c_int64, f64p] + [ctypes.c_int] * 3
            lib.ave_oracle_gemm_tn_entries.restype = ctypes.c_int
            lib.ave_oracle_threads.argtypes = []
            lib.ave_oracle_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def _bits(x) -> np.ndarray:
    """bf16 tensor / uint16 array -> contiguous numpy uint16 bit patterns."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint16:
            raise TypeError("numpy input must be uint16 bf16 bit patterns")
        return np.ascontiguousarray(x)
    import torch  # tensors only

    if x.dtype != torch.bfloat16 or x.device.type != "cpu":
        raise TypeError("tensor input must be a CPU bfloat16 tensor")
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def _shapes(q, k, v):
    if q.ndim != 4 or k.ndim != 4 or v.ndim != 4:
        raise ValueError("q, k, v must be 4-D [B, heads, S, D]")
    B, H, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    if tuple(v.shape) != tuple(k.shape) or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v shapes")
    return B, H, Hkv, Sq, Sk, D


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def threads() -> int:
    return int(_load().ave_oracle_threads())


def attn_fwd(q, k, v, causal: bool, scale: float, return_p: bool = False):
    """O [B,H,Sq,D], LSE [B,H,Sq] (and P [B,H,Sq,Sk]) in float64."""
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    B, H, Hkv, Sq, Sk, D = _shapes(qb, kb, vb)
    o = np.empty((B, H, Sq, D), np.float64)
    lse = np.empty((B, H, Sq), np.float64)
    p = np.empty((B, H, Sq, Sk), np.float64) if return_p else None
    rc = _load().ave_oracle_attn_fwd(
        _ptr(qb, ctypes.c_uint16), _ptr(kb, ctypes.c_uint16), _ptr(vb, ctypes.c_uint16),
        _ptr(o, ctypes.c_double), _ptr(lse, ctypes.c_double),
        _ptr(p, ctypes.c_double) if return_p else None,
        B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise ValueError("ave_oracle_attn_fwd rejected its arguments (rc=%d)" % rc)
    return (o, lse, p) if return_p else (o, lse)


def attn_rows(q, k, v, rows, causal: bool, scale: float):
    """Oracle values for selected rows; ``rows`` is an [n, 3] array of (b, h, i)."""
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    B, H, Hkv, Sq, Sk, D = _shapes(qb, kb, vb)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64).reshape(-1, 3))
    n = rows.shape[0]
    o = np.empty((n, D), np.float64)
    lse = np.empty((n,), np.float64)
    rc = _load().ave_oracle_attn_rows(
        _ptr(qb, ctypes.c_uint16), _ptr(kb, ctypes.c_uint16), _ptr(vb, ctypes.c_uint16),
        _ptr(rows, ctypes.c_int64), n,
        _ptr(o, ctypes.c_double), _ptr(lse, ctypes.c_double),
        B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise ValueError("ave_oracle_attn_rows rejected its arguments (rc=%d)" % rc)
    return o, lse


def bruteforce(q, k, v, causal: bool, scale: float):
    """Long-double brute force without max subtraction (tiny inputs only)."""
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    B, H, Hkv, Sq, Sk, D = _shapes(qb, kb, vb)
    o = np.empty((B, H, Sq, D), np.float64)
    lse = np.empty((B, H, Sq), np.float64)
    rc = _load().ave_oracle_bruteforce(
        _ptr(qb, ctypes.c_uint16), _ptr(kb, ctypes.c_uint16), _ptr(vb, ctypes.c_uint16),
        _ptr(o, ctypes.c_double), _ptr(lse, ctypes.c_double),
        B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise ValueError("ave_oracle_bruteforce rejected its arguments (rc=%d)" % rc)
    return o, lse


def gemm_tn(a, b):
    """C [M, N] = A [M, K] . B [N, K]^T in float64 (plain definition)."""
    ab, bb = _bits(a), _bits(b)
    if ab.ndim != 2 or bb.ndim != 2 or ab.shape[1] != bb.shape[1]:
        raise ValueError("a must be [M, K] and b [N, K]")
    M, K = ab.shape
    N = bb.shape[0]
    c = np.empty((M, N), np.float64)
    rc = _load().ave_oracle_gemm_tn(_ptr(ab, ctypes.c_uint16), _ptr(bb, ctypes.c_uint16), _ptr(c, ctypes.c_double),
                                    M, N, K)
    if rc != 0:
        raise ValueError("ave_oracle_gemm_tn rejected its arguments (rc=%d)" % rc)
    return c


def gemm_tn_entries(a, b, idx):
    """Oracle values of selected entries; ``idx`` is an [n, 2] array of (i, j)."""
    ab, bb = _bits(a), _bits(b)
    if ab.ndim != 2 or bb.ndim != 2 or ab.shape[1] != bb.shape[1]:
        raise ValueError("a must be [M, K] and b [N, K]")
    M, K = ab.shape
    N = bb.shape[0]
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int64).reshape(-1, 2))
    out = np.empty((idx.shape[0],), np.float64)
    rc = _load().ave_oracle_gemm_tn_entries(_ptr(ab, ctypes.c_uint16), _ptr(bb, ctypes.c_uint16),
                                            _ptr(idx, ctypes.c_int64), idx.shape[0], _ptr(out, ctypes.c_double),
                                            M, N, K)
    if rc != 0:
        raise ValueError("ave_oracle_gemm_tn_entries rejected its arguments (rc=%d)" % rc)
    return out
