"""Helpers shared by the GPU parity tests: run the CUDA library through its
C-ABI binding and compare against the fp64 CPU oracle."""
import numpy as np
import torch

import oracle
from paper_2604_18616_b200 import binding

O_TOL = 2e-2     # max-abs on bf16 O
LSE_TOL = 1e-3   # max-abs on fp32 LSE


def run_gpu(q, k, v, causal, scale, guard=64):
    """Run ave_attn_fwd on cuda:0 with NaN-poisoned outputs inside canary
    guard bands; returns CPU tensors (o bf16, lse fp32)."""
    dev = torch.device("cuda:0")
    B, H, Sq, D = q.shape
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    n_o, n_l = B * H * Sq * D, B * H * Sq
    o_buf = torch.full((n_o + 2 * guard,), 777.0, dtype=torch.bfloat16, device=dev)
    l_buf = torch.full((n_l + 2 * guard,), 777.0, dtype=torch.float32, device=dev)
    o = o_buf[guard:guard + n_o].view(B, H, Sq, D)
    lse = l_buf[guard:guard + n_l].view(B, H, Sq)
    o.fill_(float("nan"))
    lse.fill_(float("nan"))
    binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=causal, scale=scale)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert torch.all(o_buf[:guard] == 777.0) and torch.all(o_buf[guard + n_o:] == 777.0), "O guard band touched"
    assert torch.all(l_buf[:guard] == 777.0) and torch.all(l_buf[guard + n_l:] == 777.0), "LSE guard band touched"
    return o.cpu(), lse.cpu()


def compare(o_gpu, lse_gpu, o_ref, lse_ref, what=""):
    """Element-wise comparison against oracle arrays of the same shape."""
    og = o_gpu.double().numpy()
    lg = lse_gpu.double().numpy()
    assert not np.isnan(og).any(), what + ": NaN left in O (rows not written?)"
    assert not np.isnan(lg).any(), what + ": NaN left in LSE"
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isfinite(lg), fin), what + ": -inf pattern of LSE differs"
    assert np.all(lg[~fin] == -np.inf)
    err_o = np.abs(og - o_ref).max() if og.size else 0.0
    err_l = np.abs(lg[fin] - lse_ref[fin]).max() if fin.any() else 0.0
    assert err_o <= O_TOL, "%s: max|O - oracle| = %.4g > %g" % (what, err_o, O_TOL)
    assert err_l <= LSE_TOL, "%s: max|LSE - oracle| = %.4g > %g" % (what, err_l, LSE_TOL)
    return err_o, err_l


def check_full(q, k, v, causal, scale, what=""):
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, causal, scale)
    o, lse = run_gpu(q, k, v, causal, scale)
    return compare(o, lse, o_ref, lse_ref, what)


def check_rows(o, lse, q, k, v, rows, causal, scale, what=""):
    """Compare sampled rows (b, h, i) of a GPU result with the oracle."""
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    o_ref, lse_ref = oracle.attn_rows(q, k, v, rows, causal, scale)
    idx = (torch.from_numpy(rows[:, 0]), torch.from_numpy(rows[:, 1]), torch.from_numpy(rows[:, 2]))
    return compare(o[idx], lse[idx], o_ref, lse_ref, what)
