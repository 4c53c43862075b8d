"""The allocation-free split-KV entry point, checked against the workspace
variant and, like every other entry point, against the fp64 CPU oracle.

``ave_attn_fwd_splitkv_static`` is for callers that cannot give the library a
workspace because they may not allocate device memory at the time of the call
(all memory reserved at start-up, a latency-critical loop, an allocator owned by
the host application).  Its scratch is one array inside the library that every
call on a device shares and that keeps whatever the previous call left in it.
So the test makes two calls in a row with different shapes and key-range
counts: the second must not be disturbed by the leftovers of the first.
This file is named to be collected last.
"""
import math

import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding

import parity

pytestmark = pytest.mark.gpu


def rand_qkv(seed, B, H, Hkv, Sq, Sk, D, dev):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, H, Sq, D, generator=g).to(torch.bfloat16).to(dev)
    k = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16).to(dev)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16).to(dev)
    return q, k, v


def both_entry_points(seed, B, H, Hkv, Sq, Sk, D, causal, n_splits):
    dev = torch.device("cuda:0")
    q, k, v = rand_qkv(seed, B, H, Hkv, Sq, Sk, D, dev)
    scale = 1.0 / math.sqrt(D)
    # reference: the existing entry point with a caller-provided workspace
    o_ref, lse_ref = binding.ave_attn_fwd_splitkv(q, k, v, n_splits, causal=causal, scale=scale)
    # the allocation-free entry point; outputs pre-filled with NaN so unwritten rows show
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, H, Sq), float("nan"), dtype=torch.float32, device=dev)
    n0 = binding.launch_count()
    binding.ave_attn_fwd_splitkv_static(q, k, v, n_splits, o, lse, causal=causal, scale=scale)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert binding.launch_count() == n0 + 2          # attention kernel + merge kernel
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    assert (o.float() - o_ref.float()).abs().max().item() <= parity.O_TOL
    fin = torch.isfinite(lse_ref)
    assert torch.equal(torch.isfinite(lse), fin)
    assert (lse[fin] - lse_ref[fin]).abs().max().item() <= parity.LSE_TOL
    # both entry points against the oracle on the same inputs
    o_orc, lse_orc = oracle.attn_fwd(q.cpu(), k.cpu(), v.cpu(), causal, scale)
    parity.compare(o_ref.cpu(), lse_ref.cpu(), o_orc, lse_orc, "workspace variant")
    parity.compare(o.cpu(), lse.cpu(), o_orc, lse_orc, "built-in scratch variant")


def test_two_calls_in_a_row_share_the_built_in_scratch():
    # first call: many ranges, fills a large part of the array
    both_entry_points(1, 4, 16, 4, 3, 6000, 128, True, 24)
    # second call: other shape, fewer ranges; the array still holds the first call's partials
    both_entry_points(2, 2, 8, 8, 70, 1111, 64, False, 5)


def test_too_large_a_problem_is_rejected_before_anything_runs():
    dev = torch.device("cuda:0")
    B, H, Sq, D, n_splits = 8, 32, 256, 128, 16
    assert binding.splitkv_workspace_bytes(B, H, Sq, D, n_splits) > binding.SPLITKV_STATIC_SCRATCH_BYTES
    q = torch.zeros(B, H, Sq, D, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(B, H, 512, D, dtype=torch.bfloat16, device=dev)
    o = torch.full_like(q, 3.0)
    lse = torch.full((B, H, Sq), 3.0, dtype=torch.float32, device=dev)
    n0 = binding.launch_count()
    with pytest.raises(binding.AveAttnError) as e:
        binding.ave_attn_fwd_splitkv_static(q, kv, kv, n_splits, o, lse)
    assert e.value.status == binding.AVE_ERR_STATIC_SCRATCH
    assert "scratch" in binding.strerror(binding.AVE_ERR_STATIC_SCRATCH)
    torch.cuda.synchronize()
    assert binding.launch_count() == n0
    assert torch.all(o == 3.0) and torch.all(lse == 3.0)
