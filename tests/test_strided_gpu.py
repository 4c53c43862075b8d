"""Parity of ave_attn_fwd_strided with the fp64 oracle: the same problems as the contiguous entry point,
read and written through non-contiguous layouts (the paper's Fig. 1 (sequence, head, d) layout, a packed
QKV buffer, padded rows), without copies on the GPU side."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(B, H, Hkv, Sq, Sk, D, seed):
    w = inputs.Workload("strided", B, H, Hkv, Sq, Sk, D, True, seed)
    return inputs.make_inputs(w)


def _check(o_view, lse, q, k, v, causal, scale, what):
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, causal, scale)
    parity.compare(o_view.cpu().contiguous(), lse.cpu(), o_ref, lse_ref, what)


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [
    (2, 4, 4, 300, 300, 128, True),     # several tiles and a ragged tail
    (1, 8, 2, 257, 513, 64, True),      # GQA, Sq != Sk, D = 64
    (2, 3, 1, 128, 700, 128, False),    # non-causal, one KV head
    (1, 4, 2, 200, 330, 256, True),     # head dimension 256 (the single-sub-tile kernel)
    (1, 2, 2, 130, 130, 192, False),
])
def test_sequence_head_d_layout(B, H, Hkv, Sq, Sk, D, causal):
    """Storage (B, S, H, D) as in the paper's Fig. 1; the tensors handed over are permuted views."""
    q, k, v = _inputs(B, H, Hkv, Sq, Sk, D, 11)
    scale = D ** -0.5
    qs = q.permute(0, 2, 1, 3).contiguous().to(DEV)   # [B, Sq, H, D] storage
    ks = k.permute(0, 2, 1, 3).contiguous().to(DEV)
    vs = v.permute(0, 2, 1, 3).contiguous().to(DEV)
    os_ = torch.full((B, Sq, H, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qv, kv, vv, ov = (t.permute(0, 2, 1, 3) for t in (qs, ks, vs, os_))
    assert not qv.is_contiguous() or H == 1
    o, lse = binding.ave_attn_fwd_strided(qv, kv, vv, ov, causal=causal, scale=scale)
    _check(ov, lse, q, k, v, causal, scale, "(s,h,d) layout")


def test_packed_qkv_buffer_and_untouched_gaps():
    """One [B, S, 3, H, D] buffer holds q, k and v; O goes into a padded buffer whose gaps must stay as they were."""
    B, H, S, D = 2, 4, 384, 128
    q, k, v = _inputs(B, H, H, S, S, D, 12)
    scale = D ** -0.5
    packed = torch.stack([t.permute(0, 2, 1, 3) for t in (q, k, v)], dim=2).contiguous().to(DEV)  # [B, S, 3, H, D]
    qv, kv, vv = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    pad = 64                                            # row stride D + 64 elements
    o_store = torch.full((B, H, S, D + pad), 777.0, dtype=torch.bfloat16, device=DEV)
    ov = o_store[..., :D]
    ov.fill_(float("nan"))
    o, lse = binding.ave_attn_fwd_strided(qv, kv, vv, ov, causal=True, scale=scale)
    _check(ov, lse, q, k, v, True, scale, "packed QKV")
    assert torch.all(o_store[..., D:] == 777.0), "padding between O rows was written"


def test_strided_equals_contiguous_bitwise():
    """The same problem through both entry points gives the same bits (only the addressing differs)."""
    B, H, Hkv, S, D = 2, 8, 2, 512, 128
    q, k, v = _inputs(B, H, Hkv, S, S, D, 13)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    o1, l1 = binding.ave_attn_fwd(qd, kd, vd, causal=True)
    qs, ks, vs = (t.permute(0, 2, 1, 3).contiguous() for t in (qd, kd, vd))
    os_ = torch.empty((B, S, H, D), dtype=torch.bfloat16, device=DEV)
    o2, l2 = binding.ave_attn_fwd_strided(qs.permute(0, 2, 1, 3), ks.permute(0, 2, 1, 3), vs.permute(0, 2, 1, 3),
                                          os_.permute(0, 2, 1, 3), causal=True)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2.contiguous()) and torch.equal(l1, l2)


def test_bad_strides_are_rejected_before_any_launch():
    B, H, S, D = 1, 2, 128, 64
    x = torch.zeros((B, H, S, D), dtype=torch.bfloat16, device=DEV)
    o = torch.full_like(x, 5.0)
    lse = torch.full((B, H, S), 5.0, dtype=torch.float32, device=DEV)
    import ctypes
    L = binding.lib()
    P = lambda t: ctypes.c_void_p(t.data_ptr())
    good = (ctypes.c_longlong * 3)(H * S * D, S * D, D)
    A = lambda a: ctypes.cast(a, ctypes.c_void_p)
    n0 = binding.launch_count()

    def call(qs, ks=good, vs=good, os_=good):
        return L.ave_attn_fwd_strided(P(x), P(x), P(x), P(o), P(lse), B, H, H, S, S, D, A(qs) if qs else None,
                                      A(ks), A(vs), A(os_), 0, 1.0, None)
    assert call(None) == binding.AVE_ERR_NULL_POINTER
    assert call((ctypes.c_longlong * 3)(H * S * D, S * D, D - 8)) == binding.AVE_ERR_BAD_SHAPE      # rows overlap
    assert call((ctypes.c_longlong * 3)(0, S * D, D)) == binding.AVE_ERR_BAD_SHAPE
    assert call((ctypes.c_longlong * 3)(H * S * D, S * D, D + 4)) == binding.AVE_ERR_MISALIGNED     # not 16-byte units
    assert call(good, os_=(ctypes.c_longlong * 3)(H * S * D + 1, S * D, D)) == binding.AVE_ERR_MISALIGNED
    torch.cuda.synchronize()
    assert binding.launch_count() == n0
    assert torch.all(o == 5.0) and torch.all(lse == 5.0)
