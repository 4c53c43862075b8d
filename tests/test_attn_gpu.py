"""GPU parity: the CUDA library, called through its C ABI, against the fp64
CPU oracle on the same seeded inputs.  Tolerances: max-abs 2e-2 on bf16 O,
1e-3 on fp32 LSE."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding, inputs

import parity

pytestmark = pytest.mark.gpu


def rand_qkv(seed, B, H, Hkv, Sq, Sk, D, amp=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, H, Sq, D, generator=g) * amp).to(torch.bfloat16)
    k = (torch.randn(B, Hkv, Sk, D, generator=g) * amp).to(torch.bfloat16)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    return q, k, v


def test_config1_tiny_full_parity():
    w = inputs.get("c1_tiny")
    q, k, v = inputs.make_inputs(w)
    parity.check_full(q, k, v, w.causal, w.scale, "c1_tiny")


SHAPES = [
    # B, H, Hkv, Sq, Sk, D, causal
    (1, 1, 1, 1, 1, 64, False),
    (1, 1, 1, 1, 1, 128, True),
    (1, 2, 1, 3, 3, 64, True),
    (2, 2, 2, 63, 63, 128, False),
    (1, 2, 2, 64, 64, 64, True),
    (1, 4, 2, 65, 65, 128, True),
    (1, 2, 1, 127, 127, 64, False),
    (1, 2, 2, 128, 128, 128, True),
    (1, 3, 3, 129, 129, 128, True),
    (1, 2, 2, 129, 129, 64, False),
    (2, 4, 1, 200, 200, 128, True),
    (1, 8, 1, 257, 257, 128, True),
    (1, 2, 2, 384, 384, 64, True),
    (1, 2, 1, 300, 500, 128, False),
    (1, 4, 2, 100, 413, 128, True),    # Sq < Sk: bottom-right aligned
    (1, 2, 2, 1, 1000, 128, True),     # single query row (decode-like)
    (1, 8, 2, 7, 777, 64, True),
    (1, 2, 2, 400, 130, 128, True),    # Sq > Sk: leading rows see no key
    (1, 2, 1, 300, 40, 64, True),
    (1, 16, 2, 513, 640, 128, True),
    (3, 2, 2, 256, 1024, 64, False),
]


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", SHAPES)
def test_small_and_ragged_shapes(B, H, Hkv, Sq, Sk, D, causal):
    q, k, v = rand_qkv(B * 1000 + Sq * 7 + Sk, B, H, Hkv, Sq, Sk, D)
    parity.check_full(q, k, v, causal, 1.0 / math.sqrt(D), "shape %s" % ((B, H, Hkv, Sq, Sk, D, causal),))


def _random_shapes(n, seed):
    """Seeded random problem shapes: sizes on and around tile edges, every head grouping, both D."""
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        hkv = int(rng.choice([1, 2, 3]))
        g = int(rng.choice([1, 2, 4]))
        edge = lambda: int(rng.choice([1, 64, 127, 128, 129, 255, 256, 257, 383, 512]) + rng.integers(0, 3))
        sq, sk = (edge(), edge()) if rng.random() < 0.7 else (int(rng.integers(1, 700)), int(rng.integers(1, 900)))
        out.append((int(rng.integers(1, 3)), hkv * g, hkv, sq, sk, int(rng.choice([64, 128])), bool(rng.random() < 0.6),
                    float(rng.choice([0.05, 0.088, 0.125, 0.3]))))
    return out


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,scale", _random_shapes(24, 2024))
def test_seeded_random_shapes(B, H, Hkv, Sq, Sk, D, causal, scale):
    q, k, v = rand_qkv(Sq * 1009 + Sk, B, H, Hkv, Sq, Sk, D)
    parity.check_full(q, k, v, causal, scale, "random shape %s" % ((B, H, Hkv, Sq, Sk, D, causal, scale),))


@pytest.mark.parametrize("D", [8, 32, 40, 72, 96, 120])
@pytest.mark.parametrize("causal", [False, True])
def test_head_dimensions_other_than_64_and_128(D, causal):
    """D is any multiple of 8 up to 128: the loads zero-fill and the stores clip the columns beyond D."""
    q, k, v = rand_qkv(900 + D, 2, 4, 2, 200, 333, D)
    parity.check_full(q, k, v, causal, 1.0 / math.sqrt(D), "D = %d" % D)


def test_rows_without_keys_in_a_strided_output():
    """Causal with Sq > Sk: the leading rows see no key and are written as zeros through O's strides."""
    B, H, Sq, Sk, D = 2, 3, 400, 130, 96
    q, k, v = rand_qkv(77, B, H, H, Sq, Sk, D)
    scale = 1.0 / math.sqrt(D)
    dev = "cuda:0"
    qs, ks, vs = (t.permute(0, 2, 1, 3).contiguous().to(dev) for t in (q, k, v))   # (B, S, H, D) storage
    os_ = torch.full((B, Sq, H, D + 8), 777.0, dtype=torch.bfloat16, device=dev)      # padded rows
    ov = os_[..., :D].permute(0, 2, 1, 3)
    ov.fill_(float("nan"))
    o, lse = binding.ave_attn_fwd_strided(qs.permute(0, 2, 1, 3), ks.permute(0, 2, 1, 3), vs.permute(0, 2, 1, 3), ov,
                                          causal=True, scale=scale)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, True, scale)
    parity.compare(ov.cpu().contiguous(), lse.cpu(), o_ref, lse_ref, "strided, rows without keys")
    assert torch.all(os_[..., D:] == 777.0), "padding between O rows was written"
    assert torch.all(ov[:, :, :Sq - Sk] == 0) and torch.all(torch.isinf(lse[:, :, :Sq - Sk]))


@pytest.mark.parametrize("scale", [0.0, -0.1, 0.02, 0.3])
@pytest.mark.parametrize("causal", [False, True])
def test_scale_values_including_zero_and_negative(scale, causal):
    q, k, v = rand_qkv(5, 1, 4, 2, 200, 333, 128)
    parity.check_full(q, k, v, causal, scale, "scale %g" % scale)


def test_q_zero_closed_form_on_gpu():
    _, k, v = rand_qkv(7, 1, 4, 2, 300, 300, 128)
    q = torch.zeros(1, 4, 300, 128, dtype=torch.bfloat16)
    o, lse = parity.run_gpu(q, k, v, True, 0.1)
    i = torch.arange(300, dtype=torch.float64)
    assert torch.allclose(lse.double(), torch.log(i + 1).expand(1, 4, 300), atol=1e-3)
    pref = torch.cumsum(v.double(), dim=2) / (i + 1)[None, None, :, None]
    ref = pref.repeat_interleave(2, dim=1)
    assert (o.double() - ref).abs().max() <= parity.O_TOL


def test_one_hot_keys_select_value_rows_across_tiles():
    # keys j < D are beta * e_j; every query picks one of them.  Checks that P
    # and V pair on the key position and on the KV head (Fig. 1 assertions).
    D, Sk, Sq, H, Hkv = 128, 384, 384, 4, 2
    g = torch.Generator().manual_seed(3)
    v = torch.randn(1, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    k = torch.zeros(1, Hkv, Sk, D)
    for j in range(D):
        k[:, :, j, j] = 16.0
    q = torch.zeros(1, H, Sq, D)
    pi = [(i * 37) % min(i + 1, D) for i in range(Sq)]
    for i in range(Sq):
        q[:, :, i, pi[i]] = 16.0
    o, lse = parity.run_gpu(q.to(torch.bfloat16), k.to(torch.bfloat16), v, True, 0.25)
    for h in range(H):
        ref = v[0, h // 2][pi].double()
        assert (o[0, h].double() - ref).abs().max() <= 2 ** -7 * ref.abs().max()
    assert (lse - 64.0).abs().max() <= 1e-3


def test_peaked_and_drifting_scores_force_rescaling():
    # keys sorted by growing norm along a fixed direction: the running maximum moves in every tile
    B, H, Hkv, Sq, Sk, D = 1, 2, 1, 256, 1024, 128
    g = torch.Generator().manual_seed(9)
    q = torch.randn(B, H, Sq, D, generator=g).abs()
    k = torch.randn(B, Hkv, Sk, D, generator=g) * 0.1 + torch.linspace(0, 3, Sk)[None, None, :, None]
    v = torch.randn(B, Hkv, Sk, D, generator=g)
    parity.check_full(q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16), False, 0.05, "drift")
    parity.check_full(q.to(torch.bfloat16), k.flip(2).to(torch.bfloat16), v.to(torch.bfloat16), True, 0.05, "drift-rev")


def test_dominant_keys_with_large_values_stay_within_the_rounding_of_o():
    """Rows whose sum is dominated by one key (every 64th key scaled by 4, as in the long-context configuration)
    and values large enough that |O| passes 4, where the rounding of O to bf16 alone is up to 0.0156: the
    kernel has to add next to nothing there.  A dominant key's probability taken relative to a stale maximum
    is rounded to bf16 with an error of up to 0.2 %, which is 0.01 of such an O (a kernel that keeps the stale
    maximum there is 0.03 off on this input)."""
    B, H, Hkv, S, D = 1, 4, 2, 2048, 128
    g = torch.Generator().manual_seed(77)
    q = torch.randn(B, H, S, D, generator=g)
    k = torch.randn(B, Hkv, S, D, generator=g)
    k[:, :, ::64, :] *= 4.0
    v = torch.randn(B, Hkv, S, D, generator=g) * 1.4
    q, k, v = q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    for causal in (True, False):
        o_ref, lse_ref = oracle.attn_fwd(q, k, v, causal, scale)
        assert np.abs(o_ref).max() > 4.0          # the case is what it claims to be
        o, lse = parity.run_gpu(q, k, v, causal, scale)
        parity.compare(o, lse, o_ref, lse_ref, "dominant keys, causal=%s" % causal)


def test_gqa_equals_replicated_heads_bitwise():
    q, k, v = rand_qkv(13, 2, 8, 2, 300, 300, 128)
    o1, l1 = parity.run_gpu(q, k, v, True, 0.09)
    o2, l2 = parity.run_gpu(q, k.repeat_interleave(4, 1), v.repeat_interleave(4, 1), True, 0.09)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    assert torch.equal(l1, l2)


def test_run_to_run_bitwise_determinism():
    q, k, v = rand_qkv(17, 2, 4, 2, 640, 640, 128)
    o1, l1 = parity.run_gpu(q, k, v, True, 0.0884)
    o2, l2 = parity.run_gpu(q, k, v, True, 0.0884)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)


def test_host_buffer_entry_point_matches_device_entry_point():
    w = inputs.small_variant(inputs.get("c3_gqa_prefill"), B=1, H=8, Hkv=2, Sq=512, Sk=512)
    q, k, v = inputs.make_inputs(w)
    o_ref, l_ref = parity.run_gpu(q, k, v, True, w.scale)
    qp, kp, vp = q.pin_memory(), k.pin_memory(), v.pin_memory()
    o = torch.empty_like(q).pin_memory()
    lse = torch.empty(1, 8, 512, dtype=torch.float32).pin_memory()
    ws = torch.empty(binding.host_workspace_bytes(1, 8, 2, 512, 512, 128), dtype=torch.uint8, device="cuda:0")
    binding.ave_attn_fwd_host(qp, kp, vp, o, lse, ws, causal=True, scale=w.scale)
    torch.cuda.synchronize()
    assert torch.equal(o.view(torch.int16), o_ref.view(torch.int16)) and torch.equal(lse, l_ref)


def test_errors_launch_nothing_and_leave_outputs_alone():
    dev = torch.device("cuda:0")
    q = torch.zeros(1, 2, 128, 64, dtype=torch.bfloat16, device=dev)
    o = torch.full_like(q, 5.0)
    lse = torch.full((1, 2, 128), 5.0, device=dev)
    n0 = binding.launch_count()
    P = lambda t: t.data_ptr()
    assert binding.ave_attn_fwd_raw(P(q), P(q), P(q), P(o), P(lse), 1, 2, 2, 128, 128, 100, 0, 1.0) == binding.AVE_ERR_UNSUPPORTED_D
    assert binding.ave_attn_fwd_raw(P(q) + 2, P(q), P(q), P(o), P(lse), 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_MISALIGNED
    assert binding.ave_attn_fwd_raw(P(q), P(q), P(q), P(o), P(lse), 1, 3, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE
    assert binding.ave_attn_fwd_raw(P(q), P(q), P(q), P(o), P(lse), 1, 2, 2, 128, 128, 64, 0, float("nan")) == binding.AVE_ERR_BAD_SCALE
    torch.cuda.synchronize()
    assert binding.launch_count() == n0
    assert torch.all(o == 5.0) and torch.all(lse == 5.0)


# ---------------------------------------------------------------- full-size configs
@pytest.mark.parametrize("name,n_random", [
    ("c2_mha_prefill", 1024),
    ("c3_gqa_prefill", 1024),
    ("c4_long_context", 768),
    ("c5_wide_noncausal", 768),
    ("paper_gqa_n2048", 512),       # the paper's own evaluation shape (one KV head shared by 8 query heads)
])
def test_full_size_configs_sampled_rows(name, n_random):
    w = inputs.get(name)
    q, k, v = inputs.make_inputs(w)
    o, lse = parity.run_gpu(q, k, v, w.causal, w.scale)
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    rows = inputs.sample_rows(w, n_random)
    parity.check_rows(o, lse, q, k, v, rows, w.causal, w.scale, name)
    # property that holds at any size: softmax weights are a convex combination of V rows
    vmax = v.float().abs().amax().item()
    assert o.float().abs().max().item() <= vmax * (1 + 2 ** -7)


WIDE_SHAPES = [
    # B, H, Hkv, Sq, Sk, D, causal : head dimensions above 128 (computed with 256 output columns)
    (1, 2, 2, 1, 1, 256, True),
    (1, 2, 1, 130, 130, 256, True),
    (2, 4, 2, 257, 300, 192, True),
    (1, 3, 3, 128, 513, 256, False),
    (1, 4, 1, 300, 300, 136, True),
    (1, 2, 2, 400, 130, 200, True),     # Sq > Sk: leading rows see no key
    (1, 8, 2, 7, 777, 248, False),
]


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", WIDE_SHAPES)
def test_head_dimensions_above_128(B, H, Hkv, Sq, Sk, D, causal):
    q, k, v = rand_qkv(D * 31 + Sq, B, H, Hkv, Sq, Sk, D)
    parity.check_full(q, k, v, causal, 1.0 / math.sqrt(D), "wide head %s" % ((B, H, Hkv, Sq, Sk, D, causal),))


@pytest.mark.parametrize("name", ["d192_gqa_prefill", "d256_gqa_prefill"])
def test_wide_head_workloads_sampled_rows(name):
    """Full-size runs of the wide-head workloads: tile-edge rows of every (b, h) plus random rows, and two runs
    bit for bit equal."""
    w = inputs.get(name)
    q, k, v = inputs.make_inputs(w)
    o, lse = parity.run_gpu(q, k, v, w.causal, w.scale)
    o2, lse2 = parity.run_gpu(q, k, v, w.causal, w.scale)
    assert torch.equal(o, o2) and torch.equal(lse, lse2)
    parity.check_rows(o, lse, q, k, v, inputs.sample_rows(w, 512), w.causal, w.scale, name)
