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
_SRC_MOE = os.path.join(_HERE, "ave_oracle_moe.c")
_HDR_MOE = os.path.join(_HERE, "ave_oracle_moe.h")
_LIB = os.path.join(_HERE, "libave_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``ave_oracle.c`` with gcc into ``libave_oracle.so`` beside it."""
    newest_src = max(os.path.getmtime(f) for f in (_SRC, _HDR, _SRC_MOE, _HDR_MOE))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest_src:
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", tmp, _SRC, _SRC_MOE, "-lm"]
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
            u8p = ctypes.POINTER(ctypes.c_uint8)
            f32p = ctypes.POINTER(ctypes.c_float)
            i32p = ctypes.POINTER(ctypes.c_int32)
            lib.ave_oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
            lib.ave_oracle_e4m3_decode.restype = ctypes.c_double
            lib.ave_oracle_e4m3_encode.argtypes = [ctypes.c_float]
            lib.ave_oracle_e4m3_encode.restype = ctypes.c_uint8
            lib.ave_oracle_quant_groups.argtypes = [f32p, ctypes.c_int64, u8p, f32p]
            lib.ave_oracle_quant_groups.restype = ctypes.c_int
            moe = [u8p, f32p, u8p, f32p, u8p, f32p, i32p, f32p]
            lib.ave_oracle_moe_fwd.argtypes = moe + [f64p, u8p, f32p] + [ctypes.c_int] * 5
            lib.ave_oracle_moe_fwd.restype = ctypes.c_int
            lib.ave_oracle_moe_rows.argtypes = moe + [i64p, ctypes.c_int64, f64p] + [ctypes.c_int] * 5
            lib.ave_oracle_moe_rows.restype = ctypes.c_int
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


# ------------------------------------------------------------------ fused MoE (ave_oracle_moe.h)
def e4m3_decode(code: int) -> float:
    return float(_load().ave_oracle_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(x: float) -> int:
    return int(_load().ave_oracle_e4m3_encode(float(x)))


def quant_groups(a):
    """Quantise fp32 values in groups of 128 along the last axis: (codes uint8, scales fp32)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if a.shape[-1] % 128:
        raise ValueError("the last dimension must be a multiple of 128")
    codes = np.empty(a.shape, np.uint8)
    scales = np.empty(a.shape[:-1] + (a.shape[-1] // 128,), np.float32)
    rc = _load().ave_oracle_quant_groups(_ptr(a, ctypes.c_float), a.size // 128, _ptr(codes, ctypes.c_uint8),
                                         _ptr(scales, ctypes.c_float))
    if rc != 0:
        raise ValueError("ave_oracle_quant_groups rejected its arguments")
    return codes, scales


def _moe_args(xq, sx, w13q, s13, w2q, s2, ids, wts):
    xq, w13q, w2q = (np.ascontiguousarray(a, dtype=np.uint8) for a in (xq, w13q, w2q))
    sx, s13, s2, wts = (np.ascontiguousarray(a, dtype=np.float32) for a in (sx, s13, s2, wts))
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T, C = xq.shape
    E, F2, C2 = w13q.shape
    F = F2 // 2
    K = ids.shape[1]
    if C2 != C or w2q.shape != (E, C, F) or sx.shape != (T, C // 128) or s13.shape != (E, F2 // 128, C // 128) or \
            s2.shape != (E, C // 128, F // 128) or wts.shape != (T, K) or ids.shape[0] != T:
        raise ValueError("inconsistent MoE shapes")
    ptrs = [_ptr(xq, ctypes.c_uint8), _ptr(sx, ctypes.c_float), _ptr(w13q, ctypes.c_uint8), _ptr(s13, ctypes.c_float),
            _ptr(w2q, ctypes.c_uint8), _ptr(s2, ctypes.c_float), _ptr(ids, ctypes.c_int32), _ptr(wts, ctypes.c_float)]
    keep = (xq, sx, w13q, s13, w2q, s2, ids, wts)
    return ptrs, keep, (T, C, F, E, K)


def moe_fwd(xq, sx, w13q, s13, w2q, s2, ids, wts, return_intermediate: bool = False):
    """y [T, C] in float64 (and the requantised intermediates aq [T,K,F] uint8, sa [T,K,F/128] fp32)."""
    ptrs, keep, (T, C, F, E, K) = _moe_args(xq, sx, w13q, s13, w2q, s2, ids, wts)
    y = np.empty((T, C), np.float64)
    aq = np.empty((T, K, F), np.uint8) if return_intermediate else None
    sa = np.empty((T, K, F // 128), np.float32) if return_intermediate else None
    rc = _load().ave_oracle_moe_fwd(*ptrs, _ptr(y, ctypes.c_double),
                                    _ptr(aq, ctypes.c_uint8) if return_intermediate else None,
                                    _ptr(sa, ctypes.c_float) if return_intermediate else None, T, C, F, E, K)
    if rc != 0:
        raise ValueError("ave_oracle_moe_fwd rejected its arguments (rc=%d)" % rc)
    return (y, aq, sa) if return_intermediate else y


def moe_rows(xq, sx, w13q, s13, w2q, s2, ids, wts, tokens):
    """Oracle rows of y for selected tokens: [n, C] float64."""
    ptrs, keep, (T, C, F, E, K) = _moe_args(xq, sx, w13q, s13, w2q, s2, ids, wts)
    tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int64).reshape(-1))
    y = np.empty((tok.shape[0], C), np.float64)
    rc = _load().ave_oracle_moe_rows(*ptrs, _ptr(tok, ctypes.c_int64), tok.shape[0], _ptr(y, ctypes.c_double), T, C, F, E, K)
    if rc != 0:
        raise ValueError("ave_oracle_moe_rows rejected its arguments (rc=%d)" % rc)
    return y
