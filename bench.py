#!/usr/bin/env python
"""Benchmark of the attention-forward hot path.

  python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

One step = one ave_attn_fwd pass over one batch of the named synthetic
workload (`--workload gemm_n<size>`: one ave_gemm_bf16_tn product of square
matrices of that size, reported in its own metric).  Rank 0 prints ONE JSON line.  `value` is counted TFLOP/s
(4*B*H*Sq*Sk*D, halved when causal) over all ranks with inputs resident in
HBM; `e2e` is the same metric through the host-buffer entry point with the
host<->device copies inside the timed region; `roofline` relates the kernel's
own duration to the measured dense-bf16 tensor peak; `cpu_baseline` is the fp64
oracle timed on the host cores on a bounded row sample.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "attention fwd TFLOP/s (bf16, causal=half FLOPs)"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c2_mha_prefill"
NOMINAL_BF16_TFLOPS = 2250.0          # vendor dense bf16 figure, context only
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu captures summarised under
# profiles/ (attn_fwd_ws_current_kernel_counters.md, gemm_bf16_tn_n8192_ncu_full.md); null for workloads that were not captured.
NCU_DRAM_BYTES_PER_LAUNCH = {"c2_mha_prefill": 323.7e6, "c3_gqa_prefill": 266.9e6,
                             "c4_long_context": 311.4e6, "c5_wide_noncausal": 549.9e6, "gemm_n8192": 1109.4e6}
FALLBACK_BF16_TFLOPS = 1590.0         # earlier measurement on this machine, used when no measured file exists


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), "measured (burst, torch.matmul bf16 8192^3; the stricter of the two measured rates)", d
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback", None


# ----------------------------------------------------------------- CPU oracle leg
def oracle_sample(w, q, k, v, target_seconds):
    """Time the oracle on evenly spread rows; returns (TFLOP/s, cores, description)."""
    import numpy as np
    import oracle
    from paper_2604_18616_b200 import inputs

    def rows_for(n):
        idx = np.linspace(0, w.B * w.H * w.Sq - 1, n).astype(np.int64)
        return np.stack([idx // (w.H * w.Sq), (idx // w.Sq) % w.H, idx % w.Sq], axis=1)

    def counted_flops(rows):
        off = w.Sk - w.Sq
        vis = np.minimum(w.Sk, np.maximum(0, rows[:, 2] + 1 + off)) if w.causal else np.full(len(rows), w.Sk)
        return 4.0 * w.D * float(vis.sum())

    cores = oracle.threads()
    probe = rows_for(max(64, 8 * cores))
    t0 = time.perf_counter()
    oracle.attn_rows(q, k, v, probe, w.causal, w.scale)
    t_probe = time.perf_counter() - t0
    n = int(min(w.B * w.H * w.Sq, max(len(probe), len(probe) * target_seconds / max(t_probe, 1e-6))))
    rows = rows_for(n)
    t0 = time.perf_counter()
    oracle.attn_rows(q, k, v, rows, w.causal, w.scale)
    dt = time.perf_counter() - t0
    tf = counted_flops(rows) / dt / 1e12
    desc = "%d of %d output rows of %s, evenly spread over (b,h,i), %.1f s; FLOPs counted as 4*D per visible (query,key) pair" % (
        n, w.B * w.H * w.Sq, w.name, dt)
    return tf, cores, desc, dt


def run_reference(args):
    """The reference arm: the fp64 CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2604_18616_b200 import inputs
    w = inputs.get(args.workload)
    q, k, v = inputs.make_inputs(w)
    steps = max(1, min(args.steps, 5))
    warm = max(0, min(args.warmup, 1))
    per_step = max(2.0, min(args.cpu_seconds, 60.0 / (steps + warm)))
    for _ in range(warm):
        oracle_sample(w, q, k, v, per_step)
    tfs, total, desc, cores = [], 0.0, "", 1
    for _ in range(steps):
        tf, cores, desc, dt = oracle_sample(w, q, k, v, per_step)
        tfs.append(tf)
        total += dt
    value = sum(tfs) / len(tfs)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * total / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk, "D": w.D,
                   "causal": w.causal, "note": "each step is a bounded row sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------- clock sampler
class ClockSampler:
    """Polls SM clock and throttle reasons of one GPU through NVML while a
    timed region runs."""

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.error = None

    def _loop(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
            }
            while not self._stop.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                    for bit, name in names.items():
                        if r & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
                time.sleep(0.01)
        except Exception as e:  # NVML missing: report, do not fail the bench
            self.error = repr(e)

    def __enter__(self):
        self._thread = threading.Thread(target=self._loop, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=2.0)

    def summary(self):
        import statistics
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.error:
            out["error"] = self.error
        return out


# ------------------------------------------------------------------------ GPU leg
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2604_18616_b200 import binding, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the attention path has no CPU fallback")
    binding.lib()   # raises if the CUDA library is not built
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = inputs.get(args.workload)
    # Each rank owns an independent batch of the same shape (weak scaling, no collective on the data path).
    wr = inputs.small_variant(w, seed=w.seed + 1000 * rank) if rank > 0 else w
    q, k, v = inputs.make_inputs(wr)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    o = torch.empty_like(qd)
    lse = torch.empty((w.B, w.H, w.Sq), dtype=torch.float32, device=dev)
    flops = inputs.attn_flops(w)
    stream = torch.cuda.current_stream()

    def step():
        binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=w.causal, scale=w.scale, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    n0 = binding.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            step()
        ev1.record(stream)
        barrier()
    ms = ev0.elapsed_time(ev1)
    launches = binding.launch_count() - n0
    st, raw = binding.device_status()
    if st != binding.AVE_OK:
        raise RuntimeError("device status %d (raw %#x) after the timed region" % (st, raw))

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e_steps = max(1, args.e2e_steps)
    qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
    oh = torch.empty_like(q).pin_memory()
    lh = torch.empty((w.B, w.H, w.Sq), dtype=torch.float32).pin_memory()
    ws = torch.empty(binding.host_workspace_bytes(w.B, w.H, w.Hkv, w.Sq, w.Sk, w.D), dtype=torch.uint8, device=dev)
    for _ in range(3):
        binding.ave_attn_fwd_host(qh, kh, vh, oh, lh, ws, causal=w.causal, scale=w.scale, stream=stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        binding.ave_attn_fwd_host(qh, kh, vh, oh, lh, ws, causal=w.causal, scale=w.scale, stream=stream)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    h2d = (q.numel() + k.numel() + v.numel()) * 2
    d2h = oh.numel() * 2 + lh.numel() * 4

    t = torch.tensor([ms, e2e_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_max, e2e_ms_max = t.tolist()

    if rank == 0:
        peak, peak_kind, peaks = measured_peak()
        sustained = float(peaks["bf16_tflops_sustained"]) if peaks and "bf16_tflops_sustained" in peaks else None
        ms_per_step = ms_max / args.steps
        value = world * flops / (ms_per_step * 1e-3) / 1e12
        kernel_tf = flops / ((ms / args.steps) * 1e-3) / 1e12     # this rank's kernel, one launch per step
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk, "D": w.D,
                       "causal": w.causal, "scale": w.scale, "parallelism": "dp%d (independent batches)" % world,
                       "l2": "Q+K+V+O = %.0f MiB per step exceed the 126 MB L2; no explicit flush" % (
                           inputs.min_hbm_bytes(w) / 2 ** 20)},
            "clocks": clocks.summary(),
            "e2e": {"value": world * flops / (e2e_ms_max / e2e_steps * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "achieved": kernel_tf, "peak": peak, "unit": "TFLOP/s",
                         "frac": kernel_tf / peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(w.name),
                         "traffic_unit": "bytes per launch (ncu dram read+write)",
                         "algorithmic_hbm_bytes": inputs.min_hbm_bytes(w), "peak_kind": peak_kind,
                         "frac_of_nominal_2250": kernel_tf / NOMINAL_BF16_TFLOPS,
                         # the timed region is a long back-to-back loop under the power cap: the measured
                         # sustained matmul rate is given beside the burst one
                         "peak_sustained": sustained,
                         "frac_of_sustained": (kernel_tf / sustained) if sustained else None,
                         "flops_per_launch": flops, "kernel_us": 1e3 * ms / args.steps},
        }
        if not args.no_cpu_baseline and world == 1:
            tf, cores, desc, _ = oracle_sample(w, q, k, v, args.cpu_seconds)
            line["cpu_baseline"] = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0



# ------------------------------------------------------------------- GEMM workload
GEMM_METRIC = "gemm TFLOP/s (bf16, 2*M*N*K)"


def gemm_size(name):
    """'gemm_n8192' -> 8192 (square product, the paper's Section 9 GEMM workload)."""
    n = int(name[len("gemm_n"):])
    if n <= 0 or n % 8:
        raise ValueError("gemm_n<size>: size must be a positive multiple of 8")
    return n


def gemm_oracle_sample(a, b, target_seconds):
    """Time the fp64 oracle on evenly spread entries of C; returns (TFLOP/s, cores, description, seconds)."""
    import numpy as np
    import oracle
    M, K = a.shape
    N = b.shape[0]

    def entries(n):
        idx = np.linspace(0, M * N - 1, n).astype(np.int64)
        return np.stack([idx // N, idx % N], axis=1)

    cores = oracle.threads()
    probe = entries(max(20000, 2000 * cores))
    t0 = time.perf_counter()
    oracle.gemm_tn_entries(a, b, probe)
    t_probe = time.perf_counter() - t0
    n = int(min(M * N, max(len(probe), len(probe) * target_seconds / max(t_probe, 1e-6))))
    t0 = time.perf_counter()
    oracle.gemm_tn_entries(a, b, entries(n))
    dt = time.perf_counter() - t0
    tf = 2.0 * K * n / dt / 1e12
    desc = "%d of %d entries of C (%dx%dx%d), evenly spread, %.1f s; 2*K flops per entry" % (n, M * N, M, N, K, dt)
    return tf, cores, desc, dt


def run_gemm_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2604_18616_b200 import inputs
    n = gemm_size(args.workload)
    a, b = inputs.make_gemm_inputs(n, n, n, seed=20)
    steps = max(1, min(args.steps, 5))
    warm = max(0, min(args.warmup, 1))
    per_step = max(2.0, min(args.cpu_seconds, 60.0 / (steps + warm)))
    for _ in range(warm):
        gemm_oracle_sample(a, b, per_step)
    tfs, total, desc, cores = [], 0.0, "", 1
    for _ in range(steps):
        tf, cores, desc, dt = gemm_oracle_sample(a, b, per_step)
        tfs.append(tf)
        total += dt
    value = sum(tfs) / len(tfs)
    print(json.dumps({
        "impl": "reference", "metric": GEMM_METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * total / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "M": n, "N": n, "K": n,
                   "note": "each step is a bounded sample of the entries of C"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))
    return 0


def run_gemm(args):
    import torch
    import torch.distributed as dist
    from paper_2604_18616_b200 import binding, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the GEMM path has no CPU fallback")
    binding.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    n = gemm_size(args.workload)
    a, b = inputs.make_gemm_inputs(n, n, n, seed=20 + 1000 * rank)   # an independent product per rank
    ad, bd = a.to(dev), b.to(dev)
    c = torch.empty((n, n), dtype=torch.bfloat16, device=dev)
    flops = 2.0 * n * n * n
    stream = torch.cuda.current_stream()

    def step():
        binding.ave_gemm_bf16_tn(ad, bd, c, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    n0 = binding.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            step()
        ev1.record(stream)
        barrier()
    ms = ev0.elapsed_time(ev1)
    launches = binding.launch_count() - n0
    st, raw = binding.device_status()
    if st != binding.AVE_OK:
        raise RuntimeError("device status %d (raw %#x) after the timed region" % (st, raw))

    # ---- end to end: pinned host operands in, host result out, copies inside the timed region
    e2e_steps = max(1, args.e2e_steps)
    ah, bh = a.pin_memory(), b.pin_memory()
    ch = torch.empty((n, n), dtype=torch.bfloat16).pin_memory()

    def e2e_step():
        ad.copy_(ah, non_blocking=True)
        bd.copy_(bh, non_blocking=True)
        binding.ave_gemm_bf16_tn(ad, bd, c, stream=stream)
        ch.copy_(c, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    t = torch.tensor([ms, e2e_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_max, e2e_ms_max = t.tolist()
    if rank == 0:
        peak, peak_kind, peaks = measured_peak()
        sustained = float(peaks["bf16_tflops_sustained"]) if peaks and "bf16_tflops_sustained" in peaks else None
        ms_per_step = ms_max / args.steps
        kernel_tf = flops / ((ms / args.steps) * 1e-3) / 1e12
        line = {
            "metric": GEMM_METRIC, "value": world * flops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "M": n, "N": n, "K": n, "layout": "A [M,K], B [N,K], C [M,N] row-major",
                       "parallelism": "dp%d (independent products)" % world,
                       "l2": "A+B+C = %.0f MiB per step%s" % (3 * n * n * 2 / 2 ** 20,
                                                             " exceed the 126 MB L2; no explicit flush" if 3 * n * n * 2 > 126e6
                                                             else " fit in L2 (no flush): a cache-resident case")},
            "clocks": clocks.summary(),
            "e2e": {"value": world * flops / (e2e_ms_max / e2e_steps * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": 2 * n * n * 2, "d2h_bytes_per_step": n * n * 2, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "achieved": kernel_tf, "peak": peak, "unit": "TFLOP/s",
                         "frac": kernel_tf / peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload),
                         "traffic_unit": "bytes per launch (ncu dram read+write)",
                         "algorithmic_hbm_bytes": 3 * n * n * 2, "peak_kind": peak_kind,
                         "frac_of_nominal_2250": kernel_tf / NOMINAL_BF16_TFLOPS, "peak_sustained": sustained,
                         "frac_of_sustained": (kernel_tf / sustained) if sustained else None,
                         "flops_per_launch": flops, "kernel_us": 1e3 * ms / args.steps},
        }
        if not args.no_cpu_baseline and world == 1:
            tf, cores, desc, _ = gemm_oracle_sample(a, b, args.cpu_seconds)
            line["cpu_baseline"] = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    is_gemm = args.workload.startswith("gemm_n")
    if args.impl == "reference":
        return run_gemm_reference(args) if is_gemm else run_reference(args)
    return run_gemm(args) if is_gemm else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
