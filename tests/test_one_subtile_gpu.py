"""GPU parity of the single-sub-tile attention kernel (128-row work tiles, two CTAs per SM) against the fp64
CPU oracle: the same entry points with ``ave_attn_select_kernel(AVE_KERNEL_ONE_SUBTILE)`` in force.
Tolerances as everywhere: max-abs 2e-2 on bf16 O, 1e-3 on fp32 LSE."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding, inputs

import parity
from test_attn_gpu import SHAPES, _random_shapes, rand_qkv

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def one_subtile_kernel():
    assert binding.select_kernel(binding.KERNEL_ONE_SUBTILE) == binding.AVE_OK
    yield
    assert binding.select_kernel(binding.KERNEL_AUTO) == binding.AVE_OK


def test_selector_rejects_other_values():
    assert binding.select_kernel(3) == binding.AVE_ERR_BAD_SHAPE
    assert binding.select_kernel(-1) == binding.AVE_ERR_BAD_SHAPE


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", SHAPES)
def test_small_and_ragged_shapes(B, H, Hkv, Sq, Sk, D, causal):
    q, k, v = rand_qkv(B * 1000 + Sq * 7 + Sk, B, H, Hkv, Sq, Sk, D)
    parity.check_full(q, k, v, causal, 1.0 / math.sqrt(D), "one sub-tile, shape %s" % ((B, H, Hkv, Sq, Sk, D, causal),))


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,scale", _random_shapes(16, 4048))
def test_seeded_random_shapes(B, H, Hkv, Sq, Sk, D, causal, scale):
    q, k, v = rand_qkv(Sq * 1009 + Sk, B, H, Hkv, Sq, Sk, D)
    parity.check_full(q, k, v, causal, scale, "one sub-tile, random shape")


def test_many_tiles_per_cta_and_bitwise_repeatability():
    """More work tiles than CTAs that fit: every CTA walks several tiles; two runs agree bit for bit."""
    w = inputs.small_variant(inputs.get("c2_mha_prefill"), B=2, H=24, Hkv=24, Sq=1100, Sk=1100)
    q, k, v = inputs.make_inputs(w)
    o1, l1 = parity.run_gpu(q, k, v, w.causal, w.scale)
    o2, l2 = parity.run_gpu(q, k, v, w.causal, w.scale)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    rows = inputs.sample_rows(w, 512)
    parity.check_rows(o1, l1, q, k, v, rows, w.causal, w.scale, "one sub-tile, many tiles")


def test_other_head_dimensions_and_scales():
    for D, scale in ((40, 0.2), (96, 0.1), (128, -0.07), (64, 0.0)):
        q, k, v = rand_qkv(77 + D, 1, 4, 2, 200, 333, D)
        parity.check_full(q, k, v, True, scale, "one sub-tile, D=%d scale=%g" % (D, scale))


def test_split_kv_and_varlen_through_the_same_kernel():
    dev = torch.device("cuda:0")
    q, k, v = rand_qkv(5, 2, 8, 2, 3, 1500, 128)
    o, lse = binding.ave_attn_fwd_splitkv(q.to(dev), k.to(dev), v.to(dev), 5, causal=True, scale=0.09)
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, True, 0.09)
    parity.compare(o.cpu(), lse.cpu(), o_ref, lse_ref, "one sub-tile, split-KV")
    # variable-length batch: three sequences, token-major
    lens = [130, 1, 300]
    H, Hkv, D = 4, 2, 64
    g = torch.Generator().manual_seed(9)
    tot = sum(lens)
    qv = torch.randn(tot, H, D, generator=g).to(torch.bfloat16)
    kv = torch.randn(tot, Hkv, D, generator=g).to(torch.bfloat16)
    vv = torch.randn(tot, Hkv, D, generator=g).to(torch.bfloat16)
    cu = torch.tensor([0] + list(np.cumsum(lens)), dtype=torch.int32)
    ov, lv = binding.ave_attn_fwd_varlen(qv.to(dev), kv.to(dev), vv.to(dev), cu.to(dev), cu.to(dev), max(lens), max(lens),
                                         causal=True, scale=0.125)
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)
    for b, n in enumerate(lens):
        lo = int(cu[b])
        qs = qv[lo:lo + n].permute(1, 0, 2).unsqueeze(0).contiguous()
        ks = kv[lo:lo + n].permute(1, 0, 2).unsqueeze(0).contiguous()
        vs = vv[lo:lo + n].permute(1, 0, 2).unsqueeze(0).contiguous()
        o_ref, lse_ref = oracle.attn_fwd(qs, ks, vs, True, 0.125)
        og = ov[lo:lo + n].permute(1, 0, 2).unsqueeze(0).cpu()
        lg = lv[:, lo:lo + n].unsqueeze(0).cpu()
        parity.compare(og, lg, o_ref, lse_ref, "one sub-tile, varlen sequence %d" % b)
