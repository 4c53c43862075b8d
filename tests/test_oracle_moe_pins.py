"""Pins of the fused-MoE oracle (oracle/ave_oracle_moe.c) against things other than itself: the FP8 E4M3
format against torch's own float8_e4m3fn conversions and hand values, the block quantiser against its
definition's invariants, the layer against a numpy fp64 re-computation built on torch's dequantisation and
matmul, closed forms, and routing identities.  The paper (Section 9) names the configuration and prints no
values, so tests/golden holds no fixture for it."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import inputs


def torch_decode(codes):
    return torch.from_numpy(np.asarray(codes, dtype=np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


# ------------------------------------------------------------------------------ the format
def test_decode_all_256_codes_against_torch_and_hand_values():
    ours = np.array([oracle.e4m3_decode(c) for c in range(256)])
    ref = torch_decode(np.arange(256))
    assert np.array_equal(np.isnan(ours), np.isnan(ref))
    assert list(np.flatnonzero(np.isnan(ours))) == [0x7F, 0xFF]            # no infinities, two NaN patterns
    fin = ~np.isnan(ours)
    assert np.array_equal(ours[fin], ref[fin])
    for code, val in ((0x00, 0.0), (0x01, 2.0 ** -9), (0x07, 7 * 2.0 ** -9), (0x08, 2.0 ** -6), (0x38, 1.0), (0x3C, 1.5),
                      (0x40, 2.0), (0x7E, 448.0), (0xB8, -1.0), (0xFE, -448.0)):
        assert oracle.e4m3_decode(code) == val
    assert math.copysign(1.0, oracle.e4m3_decode(0x80)) == -1.0               # negative zero


def test_encode_round_trip_ties_and_saturation():
    for c in range(256):
        if c in (0x7F, 0xFF):
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) == c
    # ties go to the even mantissa
    assert oracle.e4m3_encode(1.0625) == 0x38          # between 1.0 (m=0) and 1.125 (m=1)
    assert oracle.e4m3_encode(1.1875) == 0x3A          # between 1.125 (m=1) and 1.25 (m=2)
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00      # between 0 and the smallest subnormal
    assert oracle.e4m3_encode(3 * 2.0 ** -10) == 0x02  # between 2^-9 (m=1) and 2*2^-9 (m=2)
    assert oracle.e4m3_encode(15.5 * 2.0 ** -10) == 0x08   # rounds up into the smallest normal
    # saturation instead of NaN / infinity
    for x in (448.0, 449.0, 464.0, 1e9, float("inf")):
        assert oracle.e4m3_encode(x) == 0x7E and oracle.e4m3_encode(-x) == 0xFE
    assert oracle.e4m3_encode(float("nan")) == 0x7F
    # against torch's conversion on random in-range values (it rounds to nearest even too)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4000) * 3, rng.uniform(-440, 440, 2000), rng.standard_normal(2000) * 0.01]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    ours = np.array([oracle.e4m3_encode(float(v)) for v in x], dtype=np.uint8)
    same = ours == ref
    # the only permitted difference is the sign bit of a value that rounds to zero
    assert np.all(same | ((ours & 0x7F) == 0) & ((ref & 0x7F) == 0))


def test_encode_is_monotonic_and_nearest():
    vals = np.array([oracle.e4m3_decode(c) for c in range(0x7F)])             # the non-negative finite values, ascending
    assert np.all(np.diff(vals) > 0)
    rng = np.random.default_rng(1)
    for x in rng.uniform(0, 448, 3000).astype(np.float32):
        got = oracle.e4m3_decode(oracle.e4m3_encode(float(x)))
        assert abs(got - float(x)) == np.min(np.abs(vals - float(x)))


# --------------------------------------------------------------------------- the quantiser
def test_block_quantiser_invariants():
    rng = np.random.default_rng(2)
    a = (rng.standard_normal((6, 256)) * rng.uniform(0.01, 30, (6, 1))).astype(np.float32)
    a[2, :128] = 0.0                                                          # an all-zero group
    a[3, 5] = 1000.0
    codes, scales = oracle.quant_groups(a)
    assert codes.shape == (6, 256) and scales.shape == (6, 2) and scales.dtype == np.float32
    amax = np.abs(a.reshape(6, 2, 128)).max(axis=2)
    expect = np.where(amax > 0, (amax / np.float32(448.0)).astype(np.float32), np.float32(1.0))
    assert np.array_equal(scales, expect)                                     # fp32 division, nothing else
    assert np.all(codes[2, :128] == 0) and scales[2, 0] == 1.0
    deq = torch_decode(codes) * np.repeat(scales.astype(np.float64), 128, axis=1)
    # the largest element of a group lands on +-448 exactly; everything is within half a step of its value
    g = np.abs(a.reshape(6, 2, 128))
    for r in range(6):
        for h in range(2):
            if amax[r, h] > 0:
                j = int(np.argmax(g[r, h]))
                assert codes[r, h * 128 + j] & 0x7F == 0x7E
    rel = np.abs(deq - a) / np.maximum(np.abs(a), 1e-30)
    big = np.abs(a) > np.repeat(scales, 128, axis=1) * 2.0 ** -6             # normal range of the scaled value
    assert rel[big].max() <= 2.0 ** -4 + 1e-6
    assert np.abs(deq - a)[~big].max() <= np.repeat(scales, 128, axis=1)[~big].max() * 2.0 ** -10 + 1e-12


# -------------------------------------------------------------------------------- the layer
def tiny(seed=3, T=5, C=256, F=128, E=3, K=2):
    w = inputs.MoeWorkload("tiny", T, C, F, E, K, seed)
    return w, [t.numpy() for t in inputs.make_moe_inputs(w)]


def numpy_moe(xq, sx, w13q, s13, w2q, s2, ids, wts):
    """Independent re-computation: torch's float8 dequantisation and cast, numpy fp64 matmul."""
    T, C = xq.shape
    E, F2, _ = w13q.shape
    F = F2 // 2
    x = torch_decode(xq) * np.repeat(sx.astype(np.float64), 128, axis=1)
    w13 = torch_decode(w13q) * np.repeat(np.repeat(s13.astype(np.float64), 128, axis=1), 128, axis=2)
    w2 = torch_decode(w2q) * np.repeat(np.repeat(s2.astype(np.float64), 128, axis=1), 128, axis=2)
    y = np.zeros((T, C))
    aq_all = np.zeros((T, ids.shape[1], F), np.uint8)
    for t in range(T):
        for k in range(ids.shape[1]):
            e = int(ids[t, k])
            h = w13[e] @ x[t]
            g, u = h[:F], h[F:]
            a = (g / (1.0 + np.exp(-g)) * u).astype(np.float32)
            amax = np.abs(a.reshape(-1, 128)).max(axis=1)
            s = np.where(amax > 0, (amax / np.float32(448.0)).astype(np.float32), np.float32(1.0))
            q = torch.from_numpy((a.reshape(-1, 128) / s[:, None]).astype(np.float32)).to(torch.float8_e4m3fn)
            aq_all[t, k] = q.view(torch.uint8).numpy().reshape(-1)
            ad = q.to(torch.float64).numpy() * s[:, None].astype(np.float64)
            y[t] += float(wts[t, k]) * (w2[e] @ ad.reshape(-1))
    return y, aq_all


def test_layer_matches_a_numpy_recomputation_with_torch_fp8():
    w, args = tiny()
    y, aq, sa = oracle.moe_fwd(*args, return_intermediate=True)
    y_ref, aq_ref = numpy_moe(*args)
    assert np.array_equal(aq & 0x7F, aq_ref & 0x7F) or np.mean(aq == aq_ref) > 0.999   # codes: bit-exact up to -0
    assert np.array_equal(aq, aq_ref) or np.all((aq == aq_ref) | ((aq & 0x7F) == 0))
    assert np.abs(y - y_ref).max() <= 1e-9 * max(1.0, np.abs(y_ref).max())
    assert np.abs(y).max() > 1e-3                                               # not a trivially zero problem


def test_closed_form_one_hot_token_and_diagonal_down_projection():
    """x = e_c0, gate weights 2, up weights 1: every a_j = silu(2); all equal, so the group scale is a/448 and every
    code is 448; W2 = 0.5 on the diagonal: y_i = w * 0.5 * silu(2) for i < F, 0 beyond."""
    T, C, F, E, K = 1, 256, 128, 2, 1
    one, two, half = 0x38, 0x40, 0x30
    xq = np.zeros((T, C), np.uint8)
    xq[0, 7] = one
    sx = np.ones((T, C // 128), np.float32)
    w13q = np.zeros((E, 2 * F, C), np.uint8)
    w13q[1, :F, 7] = two
    w13q[1, F:, 7] = one
    s13 = np.ones((E, 2 * F // 128, C // 128), np.float32)
    w2q = np.zeros((E, C, F), np.uint8)
    w2q[1, np.arange(F), np.arange(F)] = half
    s2 = np.ones((E, C // 128, F // 128), np.float32)
    ids = np.array([[1]], np.int32)
    wts = np.array([[0.75]], np.float32)
    y, aq, sa = oracle.moe_fwd(xq, sx, w13q, s13, w2q, s2, ids, wts, return_intermediate=True)
    silu2 = np.float32(2.0 / (1.0 + math.exp(-2.0)))
    assert np.all(aq == 0x7E) and sa[0, 0, 0] == np.float32(silu2 / np.float32(448.0))
    expect = 0.75 * 0.5 * 448.0 * float(sa[0, 0, 0])
    assert np.allclose(y[0, :F], expect, rtol=0, atol=1e-12) and np.all(y[0, F:] == 0)
    assert abs(expect - 0.75 * 0.5 * 1.7615941559557649) < 1e-6
    # expert 0 was not selected: nothing of it may matter
    w13q[0] = 0x7F
    y2 = oracle.moe_fwd(xq, sx, w13q, s13, w2q, s2, ids, wts)
    assert np.array_equal(y, y2)


def test_routing_identities():
    w, args = tiny(seed=5, T=6, K=3, E=4)
    xq, sx, w13q, s13, w2q, s2, ids, wts = args
    y = oracle.moe_fwd(*args)
    # the K experts of a token contribute additively with their routing weights
    parts = np.zeros_like(y)
    for k in range(3):
        parts += oracle.moe_fwd(xq, sx, w13q, s13, w2q, s2, ids[:, k:k + 1], wts[:, k:k + 1])
    assert np.abs(parts - y).max() <= 1e-12 * np.abs(y).max()
    # the order of a token's experts does not matter; tokens are independent (a permutation permutes the rows)
    y_sw = oracle.moe_fwd(xq, sx, w13q, s13, w2q, s2, ids[:, ::-1].copy(), wts[:, ::-1].copy())
    assert np.abs(y_sw - y).max() <= 1e-12 * np.abs(y).max()
    perm = np.array([3, 0, 5, 1, 4, 2])
    y_p = oracle.moe_fwd(xq[perm], sx[perm], w13q, s13, w2q, s2, ids[perm], wts[perm])
    assert np.array_equal(y_p, y[perm])
    # doubling a routing weight doubles that expert's share: y is linear in wts
    y_2 = oracle.moe_fwd(xq, sx, w13q, s13, w2q, s2, ids, (2 * wts).astype(np.float32))
    assert np.abs(y_2 - 2 * y).max() <= 1e-12 * np.abs(y).max()
    # scaling an activation group's scale by a power of two scales nothing else than x: gate and up both double
    rows = oracle.moe_rows(*args, tokens=[4, 1])
    assert np.array_equal(rows, y[[4, 1]])


def test_bad_arguments_are_rejected():
    w, args = tiny()
    bad = [a.copy() for a in args]
    bad[6][0, 0] = 99                                                           # expert id out of range
    with pytest.raises(ValueError):
        oracle.moe_fwd(*bad)
    with pytest.raises(ValueError):
        oracle.quant_groups(np.zeros((2, 100), np.float32))


def test_input_generator_produces_valid_fp8_and_routing():
    w = inputs.MoeWorkload("gen", 64, 512, 256, 8, 4, 11)
    xq, sx, w13q, s13, w2q, s2, ids, wts = inputs.make_moe_inputs(w)
    for codes in (xq, w13q, w2q):
        c = codes.numpy()
        assert not np.any((c & 0x7F) == 0x7F)                                   # no NaN pattern
        assert np.all((c.reshape(-1, 128)[:, 0] & 0x7F) == 0x7E)                # block maximum present
    assert ids.min() >= 0 and ids.max() < 8 and all(len(set(r.tolist())) == 4 for r in ids)
    assert torch.allclose(wts.sum(dim=1), torch.ones(64), atol=1e-6) and wts.min() > 0
    y = oracle.moe_fwd(*[t.numpy() for t in (xq, sx, w13q, s13, w2q, s2, ids, wts)])
    assert 0.05 < np.abs(y).mean() < 50                                         # outputs of order one
