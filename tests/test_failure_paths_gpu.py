"""Failure paths of the library, exercised without faulting or hanging the GPU.

* A bounded wait that runs out: a one-warp self-test kernel waits, with the library's own bounded
  wait and a limit of 2^16 cycles, on a barrier nobody arrives on.  It must return normally and set
  the device status word; while the word is set every kernel of the library is a no-op (outputs
  untouched) although the launch calls return AVE_OK; reading the word clears it.
* Failures injected on the host: a failing tensor-map encode and a failing launch give
  AVE_ERR_CUDA with the injected code, launch nothing and leave the outputs alone.
* The tensor-map cache and the per-device kernel preparation.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding

import parity

pytestmark = pytest.mark.gpu


def small_problem(dev, seed=5, B=1, H=4, Hkv=2, Sq=200, Sk=330, D=128):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, H, Sq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(torch.bfloat16)
    return q, k, v, q.to(dev), k.to(dev), v.to(dev)


def test_a_wait_that_runs_out_sets_the_status_word_and_later_kernels_skip():
    dev = torch.device("cuda:0")
    q, k, v, qd, kd, vd = small_problem(dev)
    scale = 1.0 / math.sqrt(q.shape[-1])
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)

    assert binding.selftest_wait_timeout(16) == binding.AVE_OK
    torch.cuda.synchronize()          # the kernel returned: no hang, no trap, the context is alive
    o = torch.full_like(qd, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device=dev)
    a = torch.randn(256, 128, device=dev).to(torch.bfloat16)
    c = torch.full((256, 256), 7.0, dtype=torch.bfloat16, device=dev)
    # launches are accepted, but the kernels return at once while the word is set
    binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=True, scale=scale)
    binding.ave_gemm_bf16_tn(a, a, c)
    torch.cuda.synchronize()
    assert torch.isnan(o.float()).all() and torch.isnan(lse).all(), "a kernel ran although the status word was set"
    assert torch.all(c == 7.0)

    st, raw = binding.device_status()
    assert st == binding.AVE_ERR_DEVICE_TIMEOUT and raw == binding.STATUS_BIT_SELFTEST
    assert "wait" in binding.strerror(st)
    st, raw = binding.device_status()                  # reading cleared it
    assert (st, raw) == (binding.AVE_OK, 0)

    binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=True, scale=scale)
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, True, scale)
    parity.compare(o.cpu(), lse.cpu(), o_ref, lse_ref, "after the status word was cleared")


@pytest.mark.parametrize("what,code", [(binding.INJECT_ENCODE_FAILURE, 1),      # CUDA_ERROR_INVALID_VALUE
                                       (binding.INJECT_LAUNCH_FAILURE, 719)])   # cudaErrorLaunchFailure
def test_injected_host_failures_report_cuda_error_and_launch_nothing(what, code):
    dev = torch.device("cuda:0")
    q, k, v, qd, kd, vd = small_problem(dev, seed=6)
    o = torch.full_like(qd, 3.0)
    lse = torch.full(q.shape[:3], 3.0, dtype=torch.float32, device=dev)
    n0 = binding.launch_count()
    assert binding.selftest_inject_failures(what, 1) == binding.AVE_OK
    try:
        with pytest.raises(binding.AveAttnError) as e:
            binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=False)
    finally:
        binding.selftest_inject_failures(what, 0)
    assert e.value.status == binding.AVE_ERR_CUDA
    assert binding.last_cuda_error() == code
    torch.cuda.synchronize()
    assert binding.launch_count() == n0
    assert torch.all(o == 3.0) and torch.all(lse == 3.0)
    # the next call is unaffected
    binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=False)
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)
    assert binding.launch_count() == n0 + 1
    o_ref, lse_ref = oracle.attn_fwd(q, k, v, False, 1.0 / math.sqrt(q.shape[-1]))
    parity.compare(o.cpu(), lse.cpu(), o_ref, lse_ref, "after an injected failure")


def test_repeated_calls_on_the_same_buffers_encode_no_tensor_maps():
    dev = torch.device("cuda:0")
    q, k, v, qd, kd, vd = small_problem(dev, seed=7, Sq=130, Sk=130)
    o = torch.empty_like(qd)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=dev)
    binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=True)
    n1 = binding.tensor_map_encodes()
    for _ in range(5):
        binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=True)
    assert binding.tensor_map_encodes() == n1
    # another output buffer is another map
    o2 = torch.empty_like(qd)
    binding.ave_attn_fwd(qd, kd, vd, o2, lse, causal=True)
    assert binding.tensor_map_encodes() == n1 + 1
    torch.cuda.synchronize()
    assert torch.equal(o, o2)
    # a different shape at the same addresses must not hit the cached entry of q (k and v still hit theirs; with at
    # most 128 query rows the single-sub-tile kernel runs, which stores O without a tensor map)
    B, H, _, D = q.shape
    q64 = qd.view(-1)[:B * H * 64 * D].view(B, H, 64, D)
    o64 = o2.view(-1)[:B * H * 64 * D].view(B, H, 64, D)
    assert q64.data_ptr() == qd.data_ptr() and o64.data_ptr() == o2.data_ptr()
    n2 = binding.tensor_map_encodes()
    binding.ave_attn_fwd(q64, kd, vd, o64, lse.view(-1)[:B * H * 64].view(B, H, 64), causal=True)
    assert n2 + 1 <= binding.tensor_map_encodes() <= n2 + 2
    o_ref, _ = oracle.attn_fwd(q64.cpu(), k, v, True, 1.0 / math.sqrt(D))
    assert np.abs(o64.cpu().double().numpy() - o_ref).max() <= parity.O_TOL
    st, raw = binding.device_status()
    assert (st, raw) == (binding.AVE_OK, 0)


def test_second_device_in_one_process():
    """Kernel attributes (dynamic shared memory) are per device: the first launch on a second GPU of the
    same process must prepare the kernel there too.  Each GPU works on its own memory only."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    outs = []
    for d in (0, 1):
        dev = torch.device("cuda", d)
        q, k, v, qd, kd, vd = small_problem(dev, seed=8)
        o, lse = binding.ave_attn_fwd(qd, kd, vd, causal=True)
        with torch.cuda.device(dev):
            st, raw = binding.device_status()
        assert (st, raw) == (binding.AVE_OK, 0)
        outs.append((o.cpu(), lse.cpu()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
