"""Parity of ave_attn_fwd_varlen with the fp64 oracle: sequences of different lengths packed without padding;
every sequence is compared, row by row, with the oracle run on that sequence alone."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_and_check(lens_q, lens_k, H, Hkv, D, causal, seed, max_pad=0):
    g = torch.Generator().manual_seed(seed)
    tq, tk = int(sum(lens_q)), int(sum(lens_k))
    q = torch.randn((tq, H, D), generator=g).to(torch.bfloat16)
    k = torch.randn((tk, Hkv, D), generator=g).to(torch.bfloat16)
    v = torch.randn((tk, Hkv, D), generator=g).to(torch.bfloat16)
    cu_q = torch.tensor(np.concatenate([[0], np.cumsum(lens_q)]), dtype=torch.int32)
    cu_k = torch.tensor(np.concatenate([[0], np.cumsum(lens_k)]), dtype=torch.int32)
    scale = 1.0 / math.sqrt(D)
    guard = 64
    o_buf = torch.full((tq + 2 * guard, H, D), 777.0, dtype=torch.bfloat16, device=DEV)
    o = o_buf[guard:guard + tq]
    o.fill_(float("nan"))
    lse = torch.full((H, tq), float("nan"), dtype=torch.float32, device=DEV)
    binding.ave_attn_fwd_varlen(q.to(DEV), k.to(DEV), v.to(DEV), cu_q.to(DEV), cu_k.to(DEV),
                                max(lens_q) + max_pad, max(lens_k) + max_pad, o=o, lse=lse, causal=causal, scale=scale)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert torch.all(o_buf[:guard] == 777.0) and torch.all(o_buf[guard + tq:] == 777.0), "rows outside the batch written"
    o_c, lse_c = o.cpu(), lse.cpu()
    for b, (sq, sk) in enumerate(zip(lens_q, lens_k)):
        if sq == 0:
            continue
        q0, k0 = int(cu_q[b]), int(cu_k[b])
        o_b = o_c[q0:q0 + sq].permute(1, 0, 2).unsqueeze(0).contiguous()          # [1, H, sq, D]
        l_b = lse_c[:, q0:q0 + sq].unsqueeze(0).contiguous()                      # [1, H, sq]
        if sk == 0:
            assert torch.all(o_b == 0) and torch.all(torch.isinf(l_b) & (l_b < 0)), "sequence %d without keys" % b
            continue
        qb = q[q0:q0 + sq].permute(1, 0, 2).unsqueeze(0).contiguous()
        kb = k[k0:k0 + sk].permute(1, 0, 2).unsqueeze(0).contiguous()
        vb = v[k0:k0 + sk].permute(1, 0, 2).unsqueeze(0).contiguous()
        o_ref, lse_ref = oracle.attn_fwd(qb, kb, vb, causal, scale)
        parity.compare(o_b, l_b, o_ref, lse_ref, "sequence %d (sq=%d, sk=%d)" % (b, sq, sk))


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("D", [64, 128, 192, 256])
def test_self_attention_lengths_on_and_off_tile_edges(causal, D):
    lens = [256, 1, 127, 300, 128, 513, 32, 129]
    _run_and_check(lens, lens, 4, 2, D, causal, 31)


def test_cross_lengths_empty_sequences_and_generous_maxima():
    lens_q = [100, 0, 257, 64, 1, 300]
    lens_k = [333, 50, 129, 0, 700, 100]     # sequence 1 has no queries, sequence 3 no keys, sequence 5 has Sq > Sk
    _run_and_check(lens_q, lens_k, 6, 3, 128, True, 32, max_pad=100)
    _run_and_check(lens_q, lens_k, 6, 3, 64, False, 33)


def test_many_short_sequences_and_other_head_dimension():
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(1, 90, size=40)]
    _run_and_check(lens, lens, 8, 1, 96, True, 34)


def test_equal_lengths_match_the_batched_entry_point_bitwise():
    B, H, Hkv, S, D = 3, 4, 2, 384, 128
    g = torch.Generator().manual_seed(35)
    q = torch.randn((B, S, H, D), generator=g).to(torch.bfloat16).to(DEV)
    k = torch.randn((B, S, Hkv, D), generator=g).to(torch.bfloat16).to(DEV)
    v = torch.randn((B, S, Hkv, D), generator=g).to(torch.bfloat16).to(DEV)
    cu = torch.arange(0, (B + 1) * S, S, dtype=torch.int32, device=DEV)
    o1, l1 = binding.ave_attn_fwd_varlen(q.view(B * S, H, D), k.view(B * S, Hkv, D), v.view(B * S, Hkv, D), cu, cu, S, S,
                                         causal=True)
    o2 = torch.empty_like(q)
    o2, l2 = binding.ave_attn_fwd_strided(q.permute(0, 2, 1, 3), k.permute(0, 2, 1, 3), v.permute(0, 2, 1, 3),
                                          o2.permute(0, 2, 1, 3), causal=True)
    torch.cuda.synchronize()
    assert torch.equal(o1.view(B, S, H, D), o2.permute(0, 2, 1, 3))
    assert torch.equal(l1.view(H, B, S).permute(1, 0, 2), l2)
