"""ctypes binding of ``libave_attn.so``: argument marshalling only.

Every function has the name and argument order of its C counterpart in
``include/ave_attn.h``; tensors are passed as their ``data_ptr()``.  Nothing
here computes: if the library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libave_attn.so")

AVE_OK = 0
AVE_ERR_NULL_POINTER = 1
AVE_ERR_BAD_SHAPE = 2
AVE_ERR_UNSUPPORTED_D = 3
AVE_ERR_MISALIGNED = 4
AVE_ERR_BAD_SCALE = 5
AVE_ERR_UNSUPPORTED_DEVICE = 6
AVE_ERR_CUDA = 7
AVE_ERR_DEVICE_TIMEOUT = 8
AVE_ERR_WORKSPACE = 9
AVE_ERR_STATIC_SCRATCH = 10
AVE_ERR_KERNEL_IMAGE = 11
INJECT_LAUNCH_FAILURE = 1
INJECT_ENCODE_FAILURE = 2
STATUS_BIT_SELFTEST = 16
SPLITKV_STATIC_SCRATCH_BYTES = 8 << 20

_lib = None


class AveAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s), cuda error %d" % (
            where, status, strerror(status), last_cuda_error()))


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built by ``paper_2604_18616_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "%s is missing: build it with `python -m paper_2604_18616_b200.build` "
                "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        L.ave_attn_fwd.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp]
        L.ave_attn_fwd.restype = ci
        L.ave_attn_fwd_strided.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, ci, cf, vp]
        L.ave_attn_fwd_strided.restype = ci
        L.ave_attn_fwd_varlen.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp]
        L.ave_attn_fwd_varlen.restype = ci
        L.ave_attn_fwd_host.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp, ctypes.c_size_t, vp]
        L.ave_attn_fwd_host.restype = ci
        L.ave_attn_host_workspace_bytes.argtypes = [ci] * 6
        L.ave_attn_host_workspace_bytes.restype = ctypes.c_size_t
        L.ave_attn_fwd_splitkv.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, ci, vp, ctypes.c_size_t, vp]
        L.ave_attn_fwd_splitkv.restype = ci
        L.ave_attn_fwd_splitkv_static.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, ci, vp]
        L.ave_attn_fwd_splitkv_static.restype = ci
        L.ave_attn_splitkv_workspace_bytes.argtypes = [ci] * 5
        L.ave_attn_splitkv_workspace_bytes.restype = ctypes.c_size_t
        L.ave_attn_splitkv_default_splits.argtypes = [ci] * 6
        L.ave_attn_splitkv_default_splits.restype = ci
        L.ave_gemm_bf16_tn.argtypes = [vp, vp, vp, ci, ci, ci, vp]
        L.ave_gemm_bf16_tn.restype = ci
        L.ave_gemm_bf16_nn.argtypes = [vp, vp, vp, ci, ci, ci, vp]
        L.ave_gemm_bf16_nn.restype = ci
        L.ave_moe_fused_fwd.argtypes = [vp] * 9 + [ci] * 5 + [vp, ctypes.c_size_t, vp]
        L.ave_moe_fused_fwd.restype = ci
        L.ave_moe_workspace_bytes.argtypes = [ci] * 5
        L.ave_moe_workspace_bytes.restype = ctypes.c_size_t
        L.ave_attn_device_status.argtypes = [ctypes.POINTER(ctypes.c_uint)]
        L.ave_attn_device_status.restype = ci
        L.ave_attn_launch_count.argtypes = []
        L.ave_attn_launch_count.restype = ctypes.c_ulonglong
        L.ave_attn_strerror.argtypes = [ci]
        L.ave_attn_strerror.restype = ctypes.c_char_p
        L.ave_attn_version.argtypes = []
        L.ave_attn_version.restype = ci
        L.ave_attn_last_cuda_error.argtypes = []
        L.ave_attn_last_cuda_error.restype = ci
        L.ave_attn_select_kernel.argtypes = [ci]
        L.ave_attn_select_kernel.restype = ci
        L.ave_attn_tensor_map_encodes.argtypes = []
        L.ave_attn_tensor_map_encodes.restype = ctypes.c_ulonglong
        L.ave_attn_selftest_register_split.argtypes = [ci]
        L.ave_attn_selftest_register_split.restype = ci
        L.ave_attn_selftest_inject_failures.argtypes = [ci, ci]
        L.ave_attn_selftest_inject_failures.restype = ci
        L.ave_attn_selftest_wait_timeout.argtypes = [ci, vp]
        L.ave_attn_selftest_wait_timeout.restype = ci
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().ave_attn_strerror(int(status)).decode()


def version() -> int:
    return int(lib().ave_attn_version())


def last_cuda_error() -> int:
    return int(lib().ave_attn_last_cuda_error())


def launch_count() -> int:
    return int(lib().ave_attn_launch_count())


KERNEL_AUTO, KERNEL_TWO_SUBTILES, KERNEL_ONE_SUBTILE = 0, 1, 2


def select_kernel(which: int) -> int:
    """0: choose per problem (default); 1: the two-sub-tile kernel; 2: the single-sub-tile kernel."""
    return int(lib().ave_attn_select_kernel(int(which)))


def tensor_map_encodes() -> int:
    return int(lib().ave_attn_tensor_map_encodes())


def selftest_register_split(regs_per_thread: int) -> int:
    return int(lib().ave_attn_selftest_register_split(int(regs_per_thread)))


def selftest_inject_failures(what: int, count: int) -> int:
    return int(lib().ave_attn_selftest_inject_failures(int(what), int(count)))


def selftest_wait_timeout(limit_cycles_log2: int = 16, stream=None) -> int:
    return int(lib().ave_attn_selftest_wait_timeout(int(limit_cycles_log2), _stream_ptr(stream)))


def device_status():
    """(status, raw word) after synchronising the device; clears the word.

    While the word is non-zero (a bounded wait inside a kernel ran out) every
    kernel of the library on that device returns without writing its outputs,
    although the launch calls keep returning AVE_OK: results since the previous
    call of this function are valid only if it returns AVE_OK."""
    raw = ctypes.c_uint(0)
    st = lib().ave_attn_device_status(ctypes.byref(raw))
    return int(st), int(raw.value)


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def ave_attn_fwd_raw(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, H, Hkv, Sq, Sk, D, causal, scale, stream_ptr=None) -> int:
    """The C call with plain integers for pointers; returns the status code."""
    return int(lib().ave_attn_fwd(
        ctypes.c_void_p(q_ptr), ctypes.c_void_p(k_ptr), ctypes.c_void_p(v_ptr),
        ctypes.c_void_p(o_ptr), ctypes.c_void_p(lse_ptr),
        B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), ctypes.c_void_p(stream_ptr)))


def ave_attn_fwd(q, k, v, o=None, lse=None, causal=False, scale=None, stream=None):
    """O, LSE = attention(q, k, v) on the tensors' CUDA device.

    q [B,H,Sq,D], k/v [B,Hkv,Sk,D]: contiguous CUDA bf16.  ``o`` (bf16) and
    ``lse`` (fp32) are allocated when not given.  Raises ``AveAttnError`` on a
    non-zero status.
    """
    for t in (q, k, v):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 4):
            raise ValueError("q, k, v must be contiguous 4-D CUDA bfloat16 tensors")
    B, H, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    if tuple(v.shape) != tuple(k.shape) or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v shapes")
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    if scale is None:
        scale = D ** -0.5
    with torch.cuda.device(q.device):
        st = lib().ave_attn_fwd(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd")
    return o, lse


def ave_attn_fwd_strided(q, k, v, o, lse=None, causal=False, scale=None, stream=None):
    """The same for strided views: q, o are [B,H,Sq,D] and k, v [B,Hkv,Sk,D] CUDA bf16 tensors with any
    batch/head/row strides (last dimension contiguous), e.g. permuted views of (B,S,H,D) storage or slices
    of a packed QKV buffer; ``o`` is written in place through its strides.  ``lse`` is contiguous fp32."""
    for t in (q, k, v, o):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 4 and t.stride(3) == 1):
            raise ValueError("q, k, v, o must be 4-D CUDA bfloat16 tensors whose last dimension is contiguous")
    B, H, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    if tuple(v.shape) != tuple(k.shape) or Bk != B or Dk != D or tuple(o.shape) != tuple(q.shape):
        raise ValueError("inconsistent q/k/v/o shapes")
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    if scale is None:
        scale = D ** -0.5
    arrs = [(ctypes.c_longlong * 3)(t.stride(0), t.stride(1), t.stride(2)) for t in (q, k, v, o)]
    with torch.cuda.device(q.device):
        st = lib().ave_attn_fwd_strided(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            B, H, Hkv, Sq, Sk, D, ctypes.cast(arrs[0], ctypes.c_void_p), ctypes.cast(arrs[1], ctypes.c_void_p),
            ctypes.cast(arrs[2], ctypes.c_void_p), ctypes.cast(arrs[3], ctypes.c_void_p),
            int(bool(causal)), float(scale), _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd_strided")
    return o, lse


def ave_attn_fwd_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, o=None, lse=None, causal=False,
                        scale=None, stream=None):
    """Variable-length batch: q [total_q,H,D], k/v [total_k,Hkv,D] contiguous CUDA bf16, cu_seqlens_* CUDA int32
    [B+1].  Returns o [total_q,H,D] bf16 and lse [H,total_q] fp32."""
    for t in (q, k, v):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 3):
            raise ValueError("q, k, v must be contiguous 3-D CUDA bfloat16 tensors")
    for t in (cu_seqlens_q, cu_seqlens_k):
        if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and t.dim() == 1):
            raise ValueError("cu_seqlens must be contiguous 1-D CUDA int32 tensors")
    total_q, H, D = q.shape
    total_k, Hkv, Dk = k.shape
    B = cu_seqlens_q.numel() - 1
    if tuple(v.shape) != tuple(k.shape) or Dk != D or cu_seqlens_k.numel() != B + 1:
        raise ValueError("inconsistent shapes")
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((H, total_q), dtype=torch.float32, device=q.device)
    if scale is None:
        scale = D ** -0.5
    with torch.cuda.device(q.device):
        st = lib().ave_attn_fwd_varlen(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            ctypes.c_void_p(cu_seqlens_q.data_ptr()), ctypes.c_void_p(cu_seqlens_k.data_ptr()),
            B, H, Hkv, int(max_sq), int(max_sk), total_q, total_k, D, int(bool(causal)), float(scale),
            _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd_varlen")
    return o, lse


def host_workspace_bytes(B, H, Hkv, Sq, Sk, D) -> int:
    return int(lib().ave_attn_host_workspace_bytes(B, H, Hkv, Sq, Sk, D))


def ave_attn_fwd_host(q, k, v, o, lse, workspace, causal=False, scale=None, stream=None):
    """Host-buffer variant: q, k, v, o, lse are CPU tensors (pinned for
    asynchronous copies), ``workspace`` a CUDA uint8 tensor of at least
    ``host_workspace_bytes`` bytes.  Results are valid after the stream has
    been synchronised."""
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    if scale is None:
        scale = D ** -0.5
    with torch.cuda.device(workspace.device):
        st = lib().ave_attn_fwd_host(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale),
            ctypes.c_void_p(workspace.data_ptr()), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
            _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd_host")
    return o, lse


def splitkv_workspace_bytes(B, H, Sq, D, n_splits) -> int:
    return int(lib().ave_attn_splitkv_workspace_bytes(B, H, Sq, D, n_splits))


def splitkv_default_splits(B, H, Hkv, Sq, Sk, D) -> int:
    return int(lib().ave_attn_splitkv_default_splits(B, H, Hkv, Sq, Sk, D))


def ave_attn_fwd_splitkv(q, k, v, n_splits, workspace=None, o=None, lse=None, causal=False, scale=None, stream=None):
    """Split-KV variant of ``ave_attn_fwd``: same tensors and result; ``workspace``
    is a CUDA uint8 tensor of at least ``splitkv_workspace_bytes`` bytes
    (allocated here when not given)."""
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    if scale is None:
        scale = D ** -0.5
    if workspace is None:
        workspace = torch.empty(max(256, splitkv_workspace_bytes(B, H, Sq, D, n_splits)), dtype=torch.uint8,
                                device=q.device)
    with torch.cuda.device(q.device):
        st = lib().ave_attn_fwd_splitkv(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), int(n_splits),
            ctypes.c_void_p(workspace.data_ptr()), ctypes.c_size_t(workspace.numel()), _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd_splitkv")
    return o, lse


def ave_attn_fwd_splitkv_static(q, k, v, n_splits, o, lse, causal=False, scale=None, stream=None):
    """Split-KV attention for callers that must not allocate device memory
    (servers that reserved all of it up front, latency-critical loops, plug-ins
    whose host owns the allocator): the scratch is an array built into the
    library, ``SPLITKV_STATIC_SCRATCH_BYTES`` per GPU.  ``o`` and ``lse`` must be
    passed in, so this wrapper allocates nothing either.  Calls sharing a
    device must not overlap on the GPU."""
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    if scale is None:
        scale = D ** -0.5
    with torch.cuda.device(q.device):
        st = lib().ave_attn_fwd_splitkv_static(
            ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()), ctypes.c_void_p(v.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
            B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), int(n_splits), _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_attn_fwd_splitkv_static")
    return o, lse


def ave_gemm_bf16_tn_raw(a_ptr, b_ptr, c_ptr, M, N, K, stream_ptr=None) -> int:
    """The C call with plain integers for pointers; returns the status code."""
    return int(lib().ave_gemm_bf16_tn(ctypes.c_void_p(a_ptr), ctypes.c_void_p(b_ptr), ctypes.c_void_p(c_ptr),
                                      M, N, K, ctypes.c_void_p(stream_ptr)))


def ave_gemm_bf16_tn(a, b, c=None, stream=None):
    """C [M, N] = a [M, K] . b [N, K]^T on the tensors' CUDA device (contiguous bf16)."""
    for t in (a, b):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 2):
            raise ValueError("a and b must be contiguous 2-D CUDA bfloat16 tensors")
    M, K = a.shape
    N, Kb = b.shape
    if Kb != K:
        raise ValueError("a is [M, K] and b is [N, K]: the K sizes differ")
    if c is None:
        c = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    with torch.cuda.device(a.device):
        st = lib().ave_gemm_bf16_tn(ctypes.c_void_p(a.data_ptr()), ctypes.c_void_p(b.data_ptr()),
                                    ctypes.c_void_p(c.data_ptr()), M, N, K, _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_gemm_bf16_tn")
    return c


def ave_gemm_bf16_nn_raw(a_ptr, b_ptr, c_ptr, M, N, K, stream_ptr=None) -> int:
    """The C call with plain integers for pointers; returns the status code."""
    return int(lib().ave_gemm_bf16_nn(ctypes.c_void_p(a_ptr), ctypes.c_void_p(b_ptr), ctypes.c_void_p(c_ptr),
                                      M, N, K, ctypes.c_void_p(stream_ptr)))


def ave_gemm_bf16_nn(a, b, c=None, stream=None):
    """C [M, N] = a [M, K] . b [K, N] on the tensors' CUDA device (contiguous bf16)."""
    for t in (a, b):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 2):
            raise ValueError("a and b must be contiguous 2-D CUDA bfloat16 tensors")
    M, K = a.shape
    Kb, N = b.shape
    if Kb != K:
        raise ValueError("a is [M, K] and b is [K, N]: the K sizes differ")
    if c is None:
        c = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    with torch.cuda.device(a.device):
        st = lib().ave_gemm_bf16_nn(ctypes.c_void_p(a.data_ptr()), ctypes.c_void_p(b.data_ptr()),
                                    ctypes.c_void_p(c.data_ptr()), M, N, K, _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_gemm_bf16_nn")
    return c


def moe_workspace_bytes(T, C, F, E, K) -> int:
    return int(lib().ave_moe_workspace_bytes(T, C, F, E, K))


def ave_moe_fused_fwd(xq, sx, w13q, s13, w2q, s2, ids, wts, y=None, workspace=None, stream=None):
    """y [T, C] bf16 = fused block-quantised FP8 MoE layer on the tensors' CUDA device.

    xq u8 [T,C], sx f32 [T,C/128], w13q u8 [E,2F,C], s13 f32 [E,2F/128,C/128], w2q u8 [E,C,F],
    s2 f32 [E,C/128,F/128], ids i32 [T,K], wts f32 [T,K]: contiguous CUDA tensors.  ``workspace`` is a CUDA uint8
    tensor of at least ``moe_workspace_bytes`` bytes (allocated here when not given)."""
    for t, dt in ((xq, torch.uint8), (w13q, torch.uint8), (w2q, torch.uint8), (sx, torch.float32), (s13, torch.float32),
                  (s2, torch.float32), (ids, torch.int32), (wts, torch.float32)):
        if not (t.is_cuda and t.dtype == dt and t.is_contiguous()):
            raise ValueError("MoE inputs must be contiguous CUDA tensors of the documented dtypes")
    T, C = xq.shape
    E, F2, C2 = w13q.shape
    F = F2 // 2
    K = ids.shape[1]
    if C2 != C or tuple(w2q.shape) != (E, C, F) or tuple(ids.shape) != (T, K) or tuple(wts.shape) != (T, K):
        raise ValueError("inconsistent MoE shapes")
    if y is None:
        y = torch.empty((T, C), dtype=torch.bfloat16, device=xq.device)
    if workspace is None:
        workspace = torch.empty(max(256, moe_workspace_bytes(T, C, F, E, K)), dtype=torch.uint8, device=xq.device)
    with torch.cuda.device(xq.device):
        st = lib().ave_moe_fused_fwd(
            ctypes.c_void_p(xq.data_ptr()), ctypes.c_void_p(sx.data_ptr()), ctypes.c_void_p(w13q.data_ptr()),
            ctypes.c_void_p(s13.data_ptr()), ctypes.c_void_p(w2q.data_ptr()), ctypes.c_void_p(s2.data_ptr()),
            ctypes.c_void_p(ids.data_ptr()), ctypes.c_void_p(wts.data_ptr()), ctypes.c_void_p(y.data_ptr()),
            T, C, F, E, K, ctypes.c_void_p(workspace.data_ptr()), ctypes.c_size_t(workspace.numel()), _stream_ptr(stream))
    if st != AVE_OK:
        raise AveAttnError(st, "ave_moe_fused_fwd")
    return y
