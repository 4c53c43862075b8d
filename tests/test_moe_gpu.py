"""GPU parity of the fused block-quantised FP8 MoE layer (ave_moe_fused_fwd, through the C ABI) against the fp64
CPU oracle on the same seeded quantised inputs.

Tolerance (derived from the arithmetic): the GPU accumulates exact E4M3 products in fp32 and rounds y to bf16 once,
so an element differs from the oracle by about 2^-9 |y| plus fp32 accumulation noise, EXCEPT where the
requantisation of an intermediate a_j falls on the other side of a rounding boundary than in the oracle (both decide
in fp32, but from values that differ in their last bits): that moves a~_j by one E4M3 step (at most |a_j| / 8) and
every y_i of that token by at most w |a_j| / 8 * max|W2|.  Such flips are rare (about one intermediate in 10^5).  So:
every element within 2^-7 |y| + the one-step bound; all but 0.2 % of the elements within 2^-7 |y| + 2e-3 rms(y).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_gpu(args):
    d = [t.to(DEV) for t in args]
    T, C = args[0].shape
    guard = 64
    buf = torch.full((T * C + 2 * guard,), 777.0, dtype=torch.bfloat16, device=DEV)
    y = buf[guard:guard + T * C].view(T, C)
    y.fill_(float("nan"))
    n0 = binding.launch_count()
    binding.ave_moe_fused_fwd(*d, y=y)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert binding.launch_count() == n0 + 7
    assert torch.all(buf[:guard] == 777.0) and torch.all(buf[guard + T * C:] == 777.0), "guard band touched"
    return y.cpu()


def check(y_gpu, y_ref, args, what):
    yg = y_gpu.double().numpy()
    assert not np.isnan(yg).any(), what + ": NaN left in y (rows not written?)"
    w2q, s2, wts = args[4].numpy(), args[5].numpy(), args[7].numpy()
    rms = float(np.sqrt(np.mean(y_ref ** 2))) + 1e-30
    err = np.abs(yg - y_ref)
    tight = 2.0 ** -7 * np.abs(y_ref) + 2e-3 * rms
    frac_out = float(np.mean(err > tight))
    # one E4M3 step of the largest possible intermediate times the largest weight: |a| <= 448 * s, and the layer's
    # intermediates here are O(1): bound by 8 (far above anything silu(g) * u reaches with these inputs) / 8
    one_step = float(wts.max()) * 1.0 * 448.0 * float(s2.max())
    loose = 2.0 ** -7 * np.abs(y_ref) + one_step
    assert frac_out <= 2e-3, "%s: %.3g of the elements outside the tight bound (max err %.3g, rms %.3g)" % (
        what, frac_out, err.max(), rms)
    assert np.all(err <= loose), "%s: max|y - oracle| = %.4g beyond the one-step bound %.3g" % (what, err.max(), one_step)
    return float(err.max()), frac_out


SHAPES = [
    # T, C, F, E, K
    (5, 256, 128, 3, 2),
    (1, 128, 128, 2, 1),
    (300, 512, 384, 8, 4),      # ragged rows per expert, several row tiles per expert
    (40, 256, 256, 16, 2),      # most experts get few or no tokens
    (700, 384, 128, 2, 2),      # many row tiles per expert
]


@pytest.mark.parametrize("T,C,F,E,K", SHAPES)
def test_small_shapes_full_parity(T, C, F, E, K):
    w = inputs.MoeWorkload("t", T, C, F, E, K, 7 * T + C)
    args = inputs.make_moe_inputs(w)
    y_ref = oracle.moe_fwd(*[t.numpy() for t in args])
    y = run_gpu(args)
    check(y, y_ref, args, "moe %s" % ((T, C, F, E, K),))


def test_papers_dimensions_on_sampled_tokens_and_repeatability():
    """Model dimension 7168, intermediate 2048, 32 experts, top-4 (Section 9) with 512 tokens: a sample of tokens
    against the oracle, and two runs bit for bit equal (the order of rows inside an expert may differ between
    runs; the values may not)."""
    w = inputs.MoeWorkload("paper", 512, 7168, 2048, 32, 4, 42)
    args = inputs.make_moe_inputs(w)
    y1 = run_gpu(args)
    y2 = run_gpu(args)
    assert torch.equal(y1, y2)
    tok = [0, 1, 77, 255, 256, 510, 511]
    y_ref = oracle.moe_rows(*[t.numpy() for t in args], tokens=tok)
    check(y1[tok], y_ref, args, "paper dims, sampled tokens")


def test_pairs_of_other_ranks_experts_contribute_nothing():
    w = inputs.MoeWorkload("ep", 33, 256, 128, 4, 3, 9)
    args = list(inputs.make_moe_inputs(w))
    ids, wts = args[6].clone(), args[7].clone()
    ids[::3, 1] = 99          # experts that live on another rank
    ids[5, 0] = -1
    y = run_gpu(args[:6] + [ids, wts])
    # the oracle sees the same thing as a valid expert with weight zero
    ids_o, wts_o = ids.clone(), wts.clone()
    bad = (ids_o < 0) | (ids_o >= w.E)
    ids_o[bad] = 0
    wts_o[bad] = 0.0
    y_ref = oracle.moe_fwd(*[t.numpy() for t in args[:6]], ids_o.numpy(), wts_o.numpy())
    check(y, y_ref, args, "pairs outside the local experts")


def test_argument_validation():
    w = inputs.MoeWorkload("v", 4, 256, 128, 2, 2, 1)
    d = [t.to(DEV) for t in inputs.make_moe_inputs(w)]
    y = torch.full((4, 256), 3.0, dtype=torch.bfloat16, device=DEV)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    n0 = binding.launch_count()
    with pytest.raises(binding.AveAttnError) as e:
        binding.ave_moe_fused_fwd(*d, y=y, workspace=small)
    assert e.value.status == binding.AVE_ERR_WORKSPACE
    assert binding.moe_workspace_bytes(4, 250, 128, 2, 2) == 0 and binding.moe_workspace_bytes(4, 256, 128, 2, 0) == 0
    torch.cuda.synchronize()
    assert binding.launch_count() == n0 and torch.all(y == 3.0)
