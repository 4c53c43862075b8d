"""GPU parity of the split-KV entry point (keys cut into ranges, partial
results merged through their log-sum-exps) against the fp64 CPU oracle and
against the single-pass entry point."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding

import parity

pytestmark = pytest.mark.gpu


def rand_qkv(seed, B, H, Hkv, Sq, Sk, D):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, H, Sq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    return q, k, v


def run_split(q, k, v, causal, scale, n_splits):
    dev = torch.device("cuda:0")
    B, H, Sq, D = q.shape
    o = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((B, H, Sq), float("nan"), dtype=torch.float32, device=dev)
    nbytes = binding.splitkv_workspace_bytes(B, H, Sq, D, n_splits)
    assert nbytes > 0
    ws = torch.full((nbytes + 512,), 0xAB, dtype=torch.uint8, device=dev)   # junk: every call must rewrite what it reads
    binding.ave_attn_fwd_splitkv(q.to(dev), k.to(dev), v.to(dev), n_splits, workspace=ws[:nbytes], o=o, lse=lse,
                                 causal=causal, scale=scale)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert torch.all(ws[nbytes:] == 0xAB), "workspace overrun"
    return o.cpu(), lse.cpu()


CASES = [
    # B, H, Hkv, Sq, Sk, D, causal, n_splits
    (2, 8, 2, 1, 4096, 128, False, 8),      # decode, GQA
    (2, 8, 2, 1, 4096, 128, True, 8),       # decode, causal (the one row sees every key)
    (1, 4, 4, 5, 1000, 64, True, 3),        # ragged key count, ranges with a masked tail
    (1, 2, 1, 64, 8269, 128, True, 16),
    (1, 2, 2, 300, 2048, 128, True, 4),     # more than one work tile per head; early ranges see nothing late
    (1, 2, 2, 17, 130, 64, False, 64),      # more ranges than key tiles: most ranges are empty
    (1, 4, 2, 33, 1500, 128, False, 1),     # a single range
]


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,n_splits", CASES)
def test_splitkv_matches_oracle_and_single_pass(B, H, Hkv, Sq, Sk, D, causal, n_splits):
    q, k, v = rand_qkv(Sq * 31 + Sk + n_splits, B, H, Hkv, Sq, Sk, D)
    scale = 1.0 / math.sqrt(D)
    o, lse = run_split(q, k, v, causal, scale, n_splits)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, causal, scale)
    parity.compare(o, lse, o_ref, lse_ref, "splitkv %s" % ((B, H, Hkv, Sq, Sk, D, causal, n_splits),))
    o1, lse1 = parity.run_gpu(q, k, v, causal, scale)
    assert (o.float() - o1.float()).abs().max() <= parity.O_TOL
    fin = torch.isfinite(lse1)
    assert torch.equal(torch.isfinite(lse), fin)
    assert (lse[fin] - lse1[fin]).abs().max() <= parity.LSE_TOL


def test_splitkv_rows_without_visible_keys():
    # Sq > Sk, causal: the first Sq - Sk rows see no key in any range
    q, k, v = rand_qkv(3, 1, 2, 2, 200, 150, 128)
    o, lse = run_split(q, k, v, True, 0.1, 2)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, True, 0.1)
    parity.compare(o, lse, o_ref, lse_ref, "splitkv Sq>Sk")
    assert torch.all(lse[:, :, :50] == float("-inf")) and torch.all(o[:, :, :50] == 0)


def test_splitkv_argument_checks():
    dev = torch.device("cuda:0")
    q = torch.zeros(1, 2, 8, 64, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(1, 2, 256, 64, dtype=torch.bfloat16, device=dev)
    assert binding.splitkv_workspace_bytes(1, 2, 8, 64, 0) == 0
    assert binding.splitkv_workspace_bytes(1, 2, 8, 64, 65) == 0
    assert binding.splitkv_workspace_bytes(1, 2, 8, 64, 4) == 4 * 16 * 65 * 4
    small = torch.empty(256, dtype=torch.uint8, device=dev)
    with pytest.raises(binding.AveAttnError) as e:
        binding.ave_attn_fwd_splitkv(q, kv, kv, 4, workspace=small)
    assert e.value.status == binding.AVE_ERR_WORKSPACE
    with pytest.raises(binding.AveAttnError) as e:
        binding.ave_attn_fwd_splitkv(q, kv, kv, 0, workspace=small)
    assert e.value.status == binding.AVE_ERR_BAD_SHAPE


PACKED = [
    # grouped-query heads with few query rows: the G heads of a KV head share work tiles
    (2, 16, 2, 1, 3000, 128, True, 4),
    (1, 8, 1, 37, 700, 64, True, 2),      # 8 * 37 = 296 rows: tiles straddle heads, causal positions wrap
    (1, 12, 4, 100, 1000, 128, True, 3),  # G = 3
    (2, 8, 2, 255, 600, 128, True, 2),
    (1, 16, 4, 5, 2048, 128, False, 8),
]


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,n_splits", PACKED)
def test_splitkv_packed_query_heads(B, H, Hkv, Sq, Sk, D, causal, n_splits):
    q, k, v = rand_qkv(Sq + Sk * 3 + H, B, H, Hkv, Sq, Sk, D)
    scale = 1.0 / math.sqrt(D)
    o, lse = run_split(q, k, v, causal, scale, n_splits)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, causal, scale)
    parity.compare(o, lse, o_ref, lse_ref, "packed %s" % ((B, H, Hkv, Sq, Sk, D, causal, n_splits),))


def test_splitkv_packed_heads_read_their_own_kv_head():
    # per-KV-head constant V: every query head must return its own group's constant
    B, H, Hkv, Sq, Sk, D = 1, 8, 4, 3, 500, 64
    q, k, _ = rand_qkv(5, B, H, Hkv, Sq, Sk, D)
    v = torch.zeros(B, Hkv, Sk, D, dtype=torch.bfloat16)
    for g in range(Hkv):
        v[:, g] = float(g + 1)
    o, _ = run_split(q, k, v, True, 0.125, 2)
    for h in range(H):
        assert torch.all(o[:, h] == float(h // 2 + 1))
