"""GPU parity of ave_gemm_bf16_tn (C = A . B^T, bf16 in, fp32 accumulation, bf16 out)
against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_18616_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def gemm_tolerance(ref, K):
    """Products of bf16 values are exact in fp32; the fp32 accumulation of K of them adds an error
    that grows like a random walk (~ K * 2^-24 for unit-variance entries), and the one rounding of
    C to bf16 costs up to 2^-9 relative.  Allowed: 2^-8 * |C| + 1e-3 * sqrt(K)."""
    return np.abs(ref) * 2.0 ** -8 + 1e-3 * np.sqrt(K)


def run_gemm(a, b, guard=64):
    dev = torch.device("cuda:0")
    M, K = a.shape
    N = b.shape[0]
    buf = torch.full((M * N + 2 * guard,), 777.0, dtype=torch.bfloat16, device=dev)
    c = buf[guard:guard + M * N].view(M, N)
    c.fill_(float("nan"))
    binding.ave_gemm_bf16_tn(a.to(dev), b.to(dev), c)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert torch.all(buf[:guard] == 777.0) and torch.all(buf[guard + M * N:] == 777.0), "guard band touched"
    return c.cpu()


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 64),        # exactly one tile, one K slice
    (128, 256, 512),       # one tile, several slices (more than the ring holds)
    (256, 512, 128),       # 2 x 2 tiles
    (1, 8, 8),             # smallest legal problem
    (127, 264, 72),        # ragged in every dimension
    (300, 1000, 200),      # ragged, several tiles
    (129, 8, 4104),        # long reduction with a ragged last slice
    (2048, 2048, 2048),    # more tiles than SMs: CTAs walk several tiles, both accumulators in use
    (2100, 2312, 264),     # the 128 x 256 tile kernel (170 tiles) with ragged edges in every dimension
    (1024, 1024, 1024),    # the 128 x 128 tile kernel, 64 tiles
])
def test_gemm_matches_oracle(M, N, K):
    a, b = inputs.make_gemm_inputs(M, N, K, seed=100 + M + N + K)
    c = run_gemm(a, b)
    cg = c.double().numpy()
    assert not np.isnan(cg).any(), "NaN left in C (entries not written?)"
    if M * N * K <= 2 ** 28:
        ref = oracle.gemm_tn(a, b)
        err = np.abs(cg - ref)
        assert (err <= gemm_tolerance(ref, K)).all(), "max err %.3g at %s" % (
            err.max(), np.unravel_index(err.argmax(), err.shape))
    else:
        rng = np.random.default_rng(7)
        edge = np.array([0, 1, 127, 128, 129, 255, 256, 257])
        ii = np.concatenate([edge[edge < M], M - 1 - edge[edge < M], rng.integers(0, M, 64)])
        jj = np.concatenate([edge[edge < N], N - 1 - edge[edge < N], rng.integers(0, N, 64)])
        idx = np.stack(np.meshgrid(ii, jj, indexing="ij"), axis=-1).reshape(-1, 2)
        ref = oracle.gemm_tn_entries(a, b, idx)
        got = cg[idx[:, 0], idx[:, 1]]
        err = np.abs(got - ref)
        assert (err <= gemm_tolerance(ref, K)).all(), "max err %.3g" % err.max()


def run_gemm_nn(a, b_kn, guard=64):
    dev = torch.device("cuda:0")
    M, K = a.shape
    N = b_kn.shape[1]
    buf = torch.full((M * N + 2 * guard,), 777.0, dtype=torch.bfloat16, device=dev)
    c = buf[guard:guard + M * N].view(M, N)
    c.fill_(float("nan"))
    binding.ave_gemm_bf16_nn(a.to(dev), b_kn.to(dev), c)
    st, raw = binding.device_status()
    assert st == binding.AVE_OK, "device status %d raw %#x" % (st, raw)
    assert torch.all(buf[:guard] == 777.0) and torch.all(buf[guard + M * N:] == 777.0), "guard band touched"
    return c.cpu()


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 64), (128, 128, 512), (1, 8, 8), (127, 264, 72), (300, 1000, 200), (129, 8, 4104),
    (1024, 1024, 1024),    # 128 x 128 tiles
    (2100, 2312, 264),     # 128 x 256 tiles, ragged
])
def test_gemm_nn_matches_oracle(M, N, K):
    """C = A . B with B stored [K, N]: the oracle's definition on the transposed copy of B."""
    a, b = inputs.make_gemm_inputs(M, N, K, seed=300 + M + N + K)
    b_kn = b.t().contiguous()          # [K, N]; b itself is [N, K]
    cg = run_gemm_nn(a, b_kn).double().numpy()
    assert not np.isnan(cg).any(), "NaN left in C (entries not written?)"
    if M * N * K <= 2 ** 28:
        ref = oracle.gemm_tn(a, b)
        err = np.abs(cg - ref)
        assert (err <= gemm_tolerance(ref, K)).all(), "max err %.3g at %s" % (
            err.max(), np.unravel_index(err.argmax(), err.shape))
    else:
        rng = np.random.default_rng(9)
        edge = np.array([0, 1, 63, 64, 65, 127, 128, 129, 255, 256, 257])
        ii = np.concatenate([edge[edge < M], M - 1 - edge[edge < M], rng.integers(0, M, 64)])
        jj = np.concatenate([edge[edge < N], N - 1 - edge[edge < N], rng.integers(0, N, 64)])
        idx = np.stack(np.meshgrid(ii, jj, indexing="ij"), axis=-1).reshape(-1, 2)
        ref = oracle.gemm_tn_entries(a, b, idx)
        err = np.abs(cg[idx[:, 0], idx[:, 1]] - ref)
        assert (err <= gemm_tolerance(ref, K)).all(), "max err %.3g" % err.max()


def test_gemm_nn_reads_b_as_k_by_n():
    """B[k, j] = 1 only at (k, j) = (3, 10): C[:, 10] = A[:, 3] and every other column is 0 — reading B
    as [N, K], or stepping through K with the wrong stride, moves or smears that column."""
    M, N, K = 40, 24, 16
    g = torch.Generator().manual_seed(12)
    a = torch.randn((M, K), generator=g).to(torch.bfloat16)
    b_kn = torch.zeros((K, N), dtype=torch.bfloat16)
    b_kn[3, 10] = 1.0
    c = run_gemm_nn(a, b_kn)
    want = torch.zeros((M, N), dtype=torch.bfloat16)
    want[:, 10] = a[:, 3]
    assert torch.equal(c, want)


def test_gemm_operands_are_not_transposed_or_swapped():
    """A non-square product with structured operands: A[i,k] = i+1 on k = 0 only, B[j,k] = j+2 on k = 0 only
    gives C[i,j] = (i+1)(j+2); any swapped or transposed operand changes the shape of that pattern."""
    M, N, K = 5, 16, 24
    a = torch.zeros((M, K), dtype=torch.bfloat16)
    b = torch.zeros((N, K), dtype=torch.bfloat16)
    a[:, 0] = torch.arange(1, M + 1, dtype=torch.float32).to(torch.bfloat16)
    b[:, 0] = torch.arange(2, N + 2, dtype=torch.float32).to(torch.bfloat16)
    c = run_gemm(a, b).double().numpy()
    want = np.outer(np.arange(1, M + 1), np.arange(2, N + 2)).astype(np.float64)
    assert np.array_equal(c, want)


def test_gemm_is_deterministic_and_full_size_sampled():
    """The paper's kind of problem (square, N(0,1)) at 4096: sampled entries against the oracle,
    and two launches give bitwise the same C."""
    n = 4096
    a, b = inputs.make_gemm_inputs(n, n, n, seed=11)
    dev = torch.device("cuda:0")
    ad, bd = a.to(dev), b.to(dev)
    c1 = binding.ave_gemm_bf16_tn(ad, bd)
    c2 = binding.ave_gemm_bf16_tn(ad, bd)
    torch.cuda.synchronize()
    assert torch.equal(c1, c2)
    rng = np.random.default_rng(3)
    idx = np.stack([rng.integers(0, n, 2048), rng.integers(0, n, 2048)], axis=1)
    ref = oracle.gemm_tn_entries(a, b, idx)
    got = c1.cpu().double().numpy()[idx[:, 0], idx[:, 1]]
    assert (np.abs(got - ref) <= gemm_tolerance(ref, n)).all()


def test_gemm_argument_errors_launch_nothing():
    dev = torch.device("cuda:0")
    a = torch.zeros((128, 64), dtype=torch.bfloat16, device=dev)
    b = torch.zeros((256, 64), dtype=torch.bfloat16, device=dev)
    c = torch.full((128, 256), 5.0, dtype=torch.bfloat16, device=dev)
    n0 = binding.launch_count()
    raw = binding.ave_gemm_bf16_tn_raw
    assert raw(0, b.data_ptr(), c.data_ptr(), 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert raw(a.data_ptr(), b.data_ptr(), c.data_ptr(), 0, 256, 64) == binding.AVE_ERR_BAD_SHAPE
    assert raw(a.data_ptr(), b.data_ptr(), c.data_ptr(), 128, 252, 64) == binding.AVE_ERR_MISALIGNED
    assert raw(a.data_ptr(), b.data_ptr(), c.data_ptr(), 128, 256, 60) == binding.AVE_ERR_MISALIGNED
    assert raw(a.data_ptr() + 2, b.data_ptr(), c.data_ptr(), 128, 256, 64) == binding.AVE_ERR_MISALIGNED
    raw_nn = binding.ave_gemm_bf16_nn_raw
    assert raw_nn(a.data_ptr(), 0, c.data_ptr(), 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert raw_nn(a.data_ptr(), b.data_ptr(), c.data_ptr(), 128, 256, -64) == binding.AVE_ERR_BAD_SHAPE
    assert raw_nn(a.data_ptr(), b.data_ptr(), c.data_ptr(), 128, 252, 64) == binding.AVE_ERR_MISALIGNED
    torch.cuda.synchronize()
    assert binding.launch_count() == n0
    assert torch.all(c == 5.0)
