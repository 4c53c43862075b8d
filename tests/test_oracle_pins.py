"""Pins for the fp64 CPU oracle: everything here runs without a GPU.

The oracle is checked against things other than itself: a long-double brute
force with no max subtraction, closed forms derived by hand from the definition
(paper Section 2: S = Q K^T, P = softmax(S), O = P V), algebraic identities of
softmax attention, and a textbook fp64 softmax + matmul from torch.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import inputs


def bf16(x):
    return torch.as_tensor(np.asarray(x), dtype=torch.float32).to(torch.bfloat16)


def rand_qkv(seed, B, H, Hkv, Sq, Sk, D, amp=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, H, Sq, D, generator=g) * amp).to(torch.bfloat16)
    k = (torch.randn(B, Hkv, Sk, D, generator=g) * amp).to(torch.bfloat16)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    return q, k, v


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("seed,B,H,Hkv,Sq,Sk,D,causal", [
    (0, 1, 1, 1, 1, 1, 1, False),
    (1, 1, 2, 2, 5, 7, 3, False),
    (2, 2, 4, 2, 7, 7, 4, True),
    (3, 1, 8, 1, 3, 9, 8, True),      # Sq < Sk: bottom-right aligned mask
    (4, 1, 4, 4, 9, 4, 5, True),      # Sq > Sk: leading rows see nothing
    (5, 2, 6, 3, 6, 11, 16, False),
    (6, 1, 8, 2, 13, 13, 2, True),
    (7, 1, 2, 1, 17, 33, 6, True),
])
def test_oracle_equals_bruteforce(seed, B, H, Hkv, Sq, Sk, D, causal):
    q, k, v = rand_qkv(seed, B, H, Hkv, Sq, Sk, D)
    scale = 0.37
    o, lse = oracle.attn_fwd(q, k, v, causal, scale)
    ob, lb = oracle.bruteforce(q, k, v, causal, scale)
    fin = np.isfinite(lb)
    assert np.array_equal(np.isfinite(lse), fin)
    assert np.all(lse[~fin] == -np.inf) and np.all(lb[~fin] == -np.inf)
    np.testing.assert_allclose(o, ob, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse[fin], lb[fin], rtol=0, atol=1e-12)


def test_rows_variant_matches_full():
    q, k, v = rand_qkv(11, 2, 4, 2, 19, 23, 8)
    o, lse = oracle.attn_fwd(q, k, v, True, 0.25)
    rows = [(b, h, i) for b in range(2) for h in range(4) for i in (0, 1, 7, 18)]
    orow, lrow = oracle.attn_rows(q, k, v, rows, True, 0.25)
    for r, (b, h, i) in enumerate(rows):
        assert np.array_equal(orow[r], o[b, h, i])
        assert lrow[r] == lse[b, h, i]


# ------------------------------------------------------------ hand closed forms
def test_three_keys_closed_form():
    # D = 1, q = 1, k = (0, 1, 2), scale = 1: softmax weights e^j / (1 + e + e^2).
    q = bf16([[[[1.0]]]])
    k = bf16([[[[0.0], [1.0], [2.0]]]])
    v = bf16([[[[1.0], [2.0], [4.0]]]])
    o, lse, p = oracle.attn_fwd(q, k, v, False, 1.0, return_p=True)
    Z = 1.0 + math.e + math.e ** 2
    assert abs(lse[0, 0, 0] - math.log(Z)) < 1e-14
    np.testing.assert_allclose(p[0, 0, 0], [1 / Z, math.e / Z, math.e ** 2 / Z], atol=1e-15)
    assert abs(o[0, 0, 0, 0] - (1 + 2 * math.e + 4 * math.e ** 2) / Z) < 1e-14


def test_scale_multiplies_scores_not_outputs():
    # q.k in {0, 2}; with scale s the weights are 1/(1+e^{2s}), e^{2s}/(1+e^{2s}).
    q = bf16([[[[1.0, 1.0]]]])
    k = bf16([[[[0.0, 0.0], [1.0, 1.0]]]])
    v = bf16([[[[0.0, 8.0], [1.0, -8.0]]]])
    for s in (0.5, -0.75, 0.0, 2.0):
        o, lse = oracle.attn_fwd(q, k, v, False, s)
        w1 = math.exp(2 * s) / (1 + math.exp(2 * s))
        np.testing.assert_allclose(o[0, 0, 0], [w1, 8.0 * (1 - w1) - 8.0 * w1], atol=1e-14)
        assert abs(lse[0, 0, 0] - math.log(1 + math.exp(2 * s))) < 1e-14


def test_transposed_operand_would_fail():
    # Q K^T with non-square, non-symmetric data: only q_i . k_j (contraction over
    # d) reproduces these scores.  Sq = 2, Sk = 3, D = 2.
    q = bf16([[[[1.0, 0.0], [0.0, 2.0]]]])
    k = bf16([[[[1.0, 3.0], [2.0, 0.0], [0.0, 1.0]]]])
    v = bf16([[[[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]]])
    o, lse = oracle.attn_fwd(q, k, v, False, 1.0)
    s = np.array([[1.0, 2.0, 0.0], [6.0, 0.0, 2.0]])
    e = np.exp(s)
    pw = e / e.sum(1, keepdims=True)
    vv = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    np.testing.assert_allclose(o[0, 0], pw @ vv, atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], np.log(e.sum(1)), atol=1e-14)


# ------------------------------------------------------------------ invariants
@pytest.mark.parametrize("causal", [False, True])
def test_softmax_rows_sum_to_one_and_mask_is_exact_zero(causal):
    q, k, v = rand_qkv(21, 1, 4, 2, 24, 37, 8, amp=2.0)
    _, lse, p = oracle.attn_fwd(q, k, v, causal, 0.5, return_p=True)
    assert np.all(p >= 0)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
    if causal:
        off = 37 - 24
        for i in range(24):
            assert np.all(p[:, :, i, i + off + 1:] == 0.0)
            assert np.all(p[:, :, i, : i + off + 1] > 0.0)


@pytest.mark.parametrize("Sq,Sk,causal", [(16, 16, False), (16, 16, True), (9, 21, True), (21, 9, True)])
def test_q_zero_gives_prefix_mean_and_log_count(Sq, Sk, causal):
    _, k, v = rand_qkv(31, 2, 4, 2, Sq, Sk, 8)
    q = torch.zeros(2, 4, Sq, 8, dtype=torch.bfloat16)
    o, lse = oracle.attn_fwd(q, k, v, causal, 0.3)
    vd = v.double().numpy()
    for i in range(Sq):
        n = min(Sk, i + 1 + (Sk - Sq)) if causal else Sk
        for h in range(4):
            g = h // 2
            if n <= 0:
                assert np.all(o[:, h, i] == 0.0) and np.all(lse[:, h, i] == -np.inf)
            else:
                np.testing.assert_allclose(o[:, h, i], vd[:, g, :n].mean(axis=1), atol=1e-13)
                np.testing.assert_allclose(lse[:, h, i], math.log(n), atol=1e-13)


def test_one_hot_keys_select_a_value_row():
    # K[j] = beta * e_j (j < D), Q[i] = beta * e_{pi(i)}; scale * beta^2 = 64 so
    # the chosen key outweighs every other by e^-64.
    D, Sk, Sq, H, Hkv = 16, 16, 16, 4, 2
    beta, scale = 16.0, 0.25
    g = torch.Generator().manual_seed(5)
    v = torch.randn(1, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    k = torch.zeros(1, Hkv, Sk, D)
    for j in range(D):
        k[:, :, j, j] = beta
    q = torch.zeros(1, H, Sq, D)
    pi = [(i * 5) % (i + 1) for i in range(Sq)]      # pi(i) <= i: visible under the causal mask
    for i in range(Sq):
        q[:, :, i, pi[i]] = beta
    o, lse = oracle.attn_fwd(q.to(torch.bfloat16), k.to(torch.bfloat16), v, True, scale)
    vd = v.double().numpy()
    for h in range(H):
        for i in range(Sq):
            np.testing.assert_allclose(o[0, h, i], vd[0, h // 2, pi[i]], atol=1e-20, rtol=1e-12)
            assert abs(lse[0, h, i] - 64.0) < 1e-12


def test_gqa_equals_replicated_mha_and_head_constants():
    q, k, v = rand_qkv(41, 2, 8, 2, 12, 15, 8)
    o, lse = oracle.attn_fwd(q, k, v, True, 0.4)
    kr = k.repeat_interleave(4, dim=1)
    vr = v.repeat_interleave(4, dim=1)
    o2, lse2 = oracle.attn_fwd(q, kr, vr, True, 0.4)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)
    # every V row of KV head g equals the constant c_g  =>  O of query head h is c_{h // G}
    vc = torch.zeros_like(v)
    vc[:, 0] = 3.0
    vc[:, 1] = -5.0
    oc, _ = oracle.attn_fwd(q, k, vc, True, 0.4)
    np.testing.assert_allclose(oc[:, :4], 3.0, atol=1e-13)
    np.testing.assert_allclose(oc[:, 4:], -5.0, atol=1e-13)


def test_key_shift_leaves_o_and_moves_lse():
    # K <- K + 1 u^T adds scale * q_i.u to every score of row i.
    q, k, v = rand_qkv(51, 1, 2, 1, 10, 14, 8)
    k = (torch.round(k.float() * 8.0) / 8.0).clamp(-3.0, 3.0).to(torch.bfloat16)   # multiples of 1/8
    u = bf16(np.array([1.0, -2.0, 0.5, 0.0, 4.0, -1.0, 2.0, 0.25]))
    k2 = (k.float() + u.float()).to(torch.bfloat16)
    assert torch.equal(k2.float(), k.float() + u.float())   # the shifted keys are exact in bf16
    o, lse = oracle.attn_fwd(q, k, v, False, 0.5)
    o2, lse2 = oracle.attn_fwd(q, k2, v, False, 0.5)
    np.testing.assert_allclose(o2, o, atol=1e-12)
    shift = 0.5 * (q.double() @ u.double()).numpy()
    np.testing.assert_allclose(lse2 - lse, shift, atol=1e-12)


def test_joint_permutation_of_keys_and_values():
    q, k, v = rand_qkv(61, 1, 4, 2, 9, 20, 8)
    perm = torch.randperm(20, generator=torch.Generator().manual_seed(1))
    o, lse = oracle.attn_fwd(q, k, v, False, 0.3)
    o2, lse2 = oracle.attn_fwd(q, k[:, :, perm], v[:, :, perm], False, 0.3)
    np.testing.assert_allclose(o2, o, atol=1e-13)
    np.testing.assert_allclose(lse2, lse, atol=1e-13)


def test_split_keys_and_merge_through_lse():
    q, k, v = rand_qkv(71, 1, 4, 2, 8, 24, 8)
    o, lse = oracle.attn_fwd(q, k, v, False, 0.6)
    o1, l1 = oracle.attn_fwd(q, k[:, :, :10], v[:, :, :10], False, 0.6)
    o2, l2 = oracle.attn_fwd(q, k[:, :, 10:], v[:, :, 10:], False, 0.6)
    lm = np.logaddexp(l1, l2)
    om = np.exp(l1 - lm)[..., None] * o1 + np.exp(l2 - lm)[..., None] * o2
    np.testing.assert_allclose(lm, lse, atol=1e-13)
    np.testing.assert_allclose(om, o, atol=1e-13)


# ---------------------------------------------------------- library cross-check
@pytest.mark.parametrize("name", ["c1_tiny"])
def test_matches_fp64_torch_softmax_matmul_on_config(name):
    w = inputs.get(name)
    q, k, v = inputs.make_inputs(w)
    o, lse = oracle.attn_fwd(q, k, v, w.causal, w.scale)
    s = (q.double() @ k.double().transpose(-1, -2)) * float(np.float32(w.scale))
    ref_o = torch.softmax(s, -1) @ v.double()
    ref_l = torch.logsumexp(s, -1)
    np.testing.assert_allclose(o, ref_o.numpy(), atol=1e-13)
    np.testing.assert_allclose(lse, ref_l.numpy(), atol=1e-13)


def test_matches_fp64_torch_with_causal_gqa_and_ragged_sizes():
    w = inputs.small_variant(inputs.get("c3_gqa_prefill"), B=2, H=8, Hkv=2, Sq=70, Sk=131, D=32)
    q, k, v = inputs.make_inputs(w)
    o, lse = oracle.attn_fwd(q, k, v, True, w.scale)
    kr = k.double().repeat_interleave(4, dim=1)
    vr = v.double().repeat_interleave(4, dim=1)
    s = (q.double() @ kr.transpose(-1, -2)) * float(np.float32(w.scale))
    i = torch.arange(70)[:, None]
    j = torch.arange(131)[None, :]
    s = s.masked_fill(j > i + (131 - 70), float("-inf"))
    np.testing.assert_allclose(o, (torch.softmax(s, -1) @ vr).numpy(), atol=1e-13)
    np.testing.assert_allclose(lse, torch.logsumexp(s, -1).numpy(), atol=1e-13)


def test_bad_arguments_are_rejected():
    q, k, v = rand_qkv(0, 1, 3, 2, 4, 4, 4)   # H % Hkv != 0
    with pytest.raises(ValueError):
        oracle.attn_fwd(q, k, v, False, 1.0)


# ------------------------------------------------------------------ GEMM oracle pins
def _bf16(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_gemm_hand_example_breaks_on_a_transposed_operand():
    # A (2x3) . B^T with B (2x3):  rows of A dotted with rows of B, by hand
    a = _bf16([[1, 2, 3], [4, 5, 6]])
    b = _bf16([[7, 8, 9], [1, 0, -1]])
    c = oracle.gemm_tn(a, b)
    assert np.array_equal(c, np.array([[50.0, -2.0], [122.0, -2.0]]))


def test_gemm_identity_and_ones():
    g = torch.Generator().manual_seed(5)
    a = torch.randn((7, 16), generator=g).to(torch.bfloat16)
    eye = torch.eye(16).to(torch.bfloat16)
    assert np.array_equal(oracle.gemm_tn(a, eye), a.double().numpy())
    ones_a = torch.ones((3, 40)).to(torch.bfloat16)
    ones_b = torch.ones((5, 40)).to(torch.bfloat16)
    assert np.array_equal(oracle.gemm_tn(ones_a, ones_b), np.full((3, 5), 40.0))


def test_gemm_bilinear_under_exact_scaling_and_matches_numpy():
    g = torch.Generator().manual_seed(6)
    a = torch.randn((33, 72), generator=g).to(torch.bfloat16)
    b = torch.randn((19, 72), generator=g).to(torch.bfloat16)
    c = oracle.gemm_tn(a, b)
    a4 = (a.float() * 4).to(torch.bfloat16)      # exact in bf16
    bh = (b.float() * 0.5).to(torch.bfloat16)
    np.testing.assert_allclose(oracle.gemm_tn(a4, bh), 2.0 * c, rtol=0, atol=0)
    ref = a.double().numpy() @ b.double().numpy().T  # the library routine, fp64
    np.testing.assert_allclose(c, ref, rtol=1e-13, atol=1e-13)
    idx = np.array([[0, 0], [32, 18], [5, 7]])
    np.testing.assert_array_equal(oracle.gemm_tn_entries(a, b, idx), c[idx[:, 0], idx[:, 1]])
