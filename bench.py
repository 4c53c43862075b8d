#!/usr/bin/env python
"""Benchmark of the attention-forward hot path.

  python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]
                  [--legs all|none|NAME,NAME...] [--scaling weak|strong] [--plan-only]

One step = one pass of the hot path (one ``ave_attn_fwd`` launch) over one batch of the named synthetic
workload; the default is the largest single-GPU prefill configuration.  Rank 0 prints ONE JSON line:

* ``value``: counted TFLOP/s (4*B*H*Sq*Sk*D, halved when causal) over all ranks, inputs resident in HBM, exactly
  K launches between two CUDA events on the launching stream, max over ranks;
* ``e2e``: the same metric through the host-buffer entry point, host<->device copies inside the timed region;
* ``roofline``: the kernel's own duration against the measured dense-bf16 tensor peak;
* ``cpu_baseline``: the fp64 oracle timed on the host cores on a bounded row sample of the same workload; the GPU
  result of a NaN-poisoned launch (outside the timed region) is compared with those oracle rows, so the line
  carries the parity errors of the very process that produced the number;
* ``per_workload`` (1 GPU only): one record per further workload (the five configurations, the paper's own shape
  at its five lengths, split-KV decode shapes, square matrix products), each timed the same way with K launches
  and checked against oracle rows the same way.

``--workload gemm_n<size>`` / ``decode_*`` make a matrix product / a split-KV decode shape the headline (used for
profiler captures of those kernels).  With ``--gpus N`` and no torchrun environment the script starts the N ranks
itself.  ``--impl reference`` times the CPU oracle alone.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "attention fwd TFLOP/s (bf16, causal=half FLOPs)"
GEMM_METRIC = "gemm TFLOP/s (bf16, 2*M*N*K)"
MOE_METRIC = "fused MoE TFLOP/s (fp8 e4m3 block-quantised, 2*T*K*(2F*C + C*F))"
FP8_OVER_BF16 = 2.0                   # nominal ratio of the dense fp8 and bf16 tensor peaks (4.5 / 2.25 PFLOP/s)
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c4_long_context"
NOMINAL_BF16_TFLOPS = 2250.0          # vendor dense bf16 figure, context only
FALLBACK_BF16_TFLOPS = 1590.0         # earlier measurements on this machine, used when no measured file exists
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126e6
PER_WORKLOAD_DEFAULT = [
    "c1_tiny", "c2_mha_prefill", "c3_gqa_prefill", "c4_long_context", "c5_wide_noncausal",
    "paper_gqa_n1024", "paper_gqa_n2048", "paper_gqa_n4096", "paper_gqa_n8192", "paper_gqa_n16384",
    "d192_gqa_prefill", "d256_gqa_prefill",
    "decode_mha_b8_k8192", "decode_gqa_b8_k16384", "decode_gqa_b1_k65536", "decode_gqa_b64_k4096",
    "gemm_n4096", "gemm_n8192", "gemm_n16384",
    "moe_t4096", "moe_t16384",
]
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from profiler captures of the
# kernel as committed; a workload whose kernel has changed since its capture is absent (reported as null).
NCU_DRAM_BYTES_PER_LAUNCH = {
    "c2_mha_prefill": 325_227_136,        # profiles/attn_fwd_ws_c2_mha_prefill_ncu.md
    "c3_gqa_prefill": 266_534_272,        # profiles/attn_fwd_ws_c3_gqa_prefill_ncu.md
    "c4_long_context": 309_833_600,       # profiles/attn_fwd_ws_c4_long_context_ncu.md
    "c5_wide_noncausal": 558_852_480,     # profiles/attn_fwd_ws_c5_wide_noncausal_ncu.md
    "d256_gqa_prefill": 303_363_968,      # profiles/attn_fwd_1t_d256_gqa_prefill_ncu.md
    "decode_mha_b8_k8192": 1_078_524_644, # profiles/attn_fwd_1t_decode_mha_b8_k8192_ncu.md
    "gemm_n8192": 1_096_847_744,          # profiles/gemm_bf16_n8192_ncu.md
}
# Unit rates measured on this part (SM clocks per instruction): one M128xN128xK16 bf16 tcgen05.mma takes 64 clk,
# an N = 64 one 47 clk; the exponential unit delivers 16 results per clock per SM.
MMA_CLK_N128, MMA_CLK_N64, EX2_PER_CLK, N_SMS = 64.0, 47.0, 16.0, 148


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--legs", default="all", help="per_workload records: all, none, or a comma-separated list")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: weak = an independent batch per rank; strong = the one batch sharded over ranks")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the headline's oracle sample")
    ap.add_argument("--leg-cpu-seconds", type=float, default=1.5, help="target oracle time of a per_workload record")
    ap.add_argument("--sustain-seconds", type=float, default=1.5,
                    help="length of the extra back-to-back loop that shows the rate under the power cap (0: skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel", type=int, default=0, choices=[0, 1, 2],
                    help="attention kernel: 0 chosen per problem (default), 1 two sub-tiles per CTA, 2 one sub-tile per CTA")
    ap.add_argument("--plan-only", action="store_true",
                    help="start the ranks, print which rank runs what, and exit (gloo on a box without GPUs)")
    return ap.parse_args(argv)


def measured_peaks():
    """(bf16 burst TFLOP/s, sustained or None, HBM GB/s, description)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return (float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]) if "bf16_tflops_sustained" in d else None,
                float(d["hbm_gbs"]), "measured on this pool (burst torch.matmul bf16 8192^3; copy bandwidth)")
    except Exception:
        return FALLBACK_BF16_TFLOPS, None, FALLBACK_HBM_GBS, "fallback"


def workload_config(w):
    """The `config` object of a JSON line: the same for the GPU arm and the oracle arm."""
    return {"workload": w.name, "B": w.B, "H": w.H, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk, "D": w.D,
            "causal": w.causal, "scale": w.scale}


# ------------------------------------------------------------------- clock sampler
class ClockSampler:
    """SM clock and throttle reasons of one GPU through NVML.  NVML is initialised and a first sample taken
    before the timed region starts; a thread then polls every 2 ms until stopped, and `sample()` lets the
    timing code add a sample at a moment it knows the GPU to be busy."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, pci_bus_id=None):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz, self.error, self._h, self._nv = None, None, None, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml as nv
            nv.nvmlInit()
            self._nv = nv
            # CUDA ordinals follow CUDA_VISIBLE_DEVICES, NVML indices do not: look the GPU up by its bus address
            try:
                self._h = nv.nvmlDeviceGetHandleByPciBusId(pci_bus_id.encode()) if pci_bus_id else None
            except Exception:
                self._h = None
            if self._h is None:
                self._h = nv.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(self._h, nv.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report, do not fail the bench
            self.error = repr(e)

    def sample(self):
        if self._h is None:
            return
        nv = self._nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
            self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
        except Exception as e:
            self.error = repr(e)

    def _loop(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.002)

    def __enter__(self):
        self.samples, self.reasons, self.power = [], set(), []
        self._stop.clear()
        self._thread = threading.Thread(target=self._loop, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=2.0)

    def summary(self):
        import statistics
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "reasons": sorted(self.reasons), "samples": len(self.samples),
               "power_w_max": max(self.power) if self.power else None}
        if self.error:
            out["error"] = self.error
        return out


def timed_launches(torch, stream, step, n, clocks, barrier=None):
    """Exactly n calls of `step` between two CUDA events on `stream`; returns milliseconds."""
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with clocks:
        (barrier or torch.cuda.synchronize)()
        ev0.record(stream)
        for i in range(n):
            step(i)
        ev1.record(stream)
        clocks.sample()               # the queue is still draining: the GPU is under load now
        (barrier or torch.cuda.synchronize)()
    return ev0.elapsed_time(ev1)


def rotation_sets(bytes_per_set):
    """Input sets to rotate over so that consecutive launches do not find their inputs in L2."""
    if bytes_per_set >= 2 * L2_BYTES:
        return 1
    return int(min(32, max(2, -(-int(2.2 * L2_BYTES) // max(1, bytes_per_set)))))


# ----------------------------------------------------------------- CPU oracle legs
def attention_rows_for_check(w, n_random):
    from paper_2604_18616_b200 import inputs
    import numpy as np
    rows = np.asarray(inputs.sample_rows(w, n_random), dtype=np.int64).reshape(-1, 3)
    return rows


def counted_flops_of_rows(w, rows):
    import numpy as np
    off = w.Sk - w.Sq
    vis = np.minimum(w.Sk, np.maximum(0, rows[:, 2] + 1 + off)) if w.causal else np.full(len(rows), w.Sk)
    return 4.0 * w.D * float(vis.sum())


def cpu_baseline_attention(w, q, k, v, target_seconds, o_gpu=None, lse_gpu=None, spread=True):
    """The CPU-baseline leg: the oracle, as it stands, timed on a bounded sample of output rows of the workload.
    When the GPU result is given, the oracle's rows are also compared with it (max-abs errors)."""
    import numpy as np
    import oracle
    total_rows = w.B * w.H * w.Sq

    def spread_rows(n):
        idx = np.linspace(0, total_rows - 1, n).astype(np.int64)
        return np.stack([idx // (w.H * w.Sq), (idx // w.Sq) % w.H, idx % w.Sq], axis=1)

    cores = oracle.threads()
    probe = spread_rows(min(total_rows, max(64, 8 * cores)))
    t0 = time.perf_counter()
    oracle.attn_rows(q, k, v, probe, w.causal, w.scale)
    t_probe = time.perf_counter() - t0
    n = int(min(total_rows, max(len(probe), len(probe) * target_seconds / max(t_probe, 1e-6))))
    if spread:
        rows = spread_rows(n)
        what = "evenly spread over (b,h,i)"
    else:   # tile-edge rows of every (b, h) plus random rows
        edge = attention_rows_for_check(w, 0)
        rows = attention_rows_for_check(w, max(64, n - len(edge)))
        what = "tile-edge rows of every (b,h) plus random rows"
    t0 = time.perf_counter()
    o_ref, lse_ref = oracle.attn_rows(q, k, v, rows, w.causal, w.scale)
    dt = time.perf_counter() - t0
    out = {"value": counted_flops_of_rows(w, rows) / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "%d of %d output rows of %s, %s, %.1f s; FLOPs counted as 4*D per visible (query,key) pair" % (
               len(rows), total_rows, w.name, what, dt),
           "seconds": dt}
    if o_gpu is not None:
        og = o_gpu[rows[:, 0], rows[:, 1], rows[:, 2]].double().numpy()
        lg = lse_gpu[rows[:, 0], rows[:, 1], rows[:, 2]].double().numpy()
        fin = np.isfinite(lse_ref)
        out["parity"] = {
            "rows": int(len(rows)),
            "max_abs_o": float(np.nanmax(np.abs(og - o_ref))) if og.size else 0.0,
            "max_abs_lse": float(np.abs(lg[fin] - lse_ref[fin]).max()) if fin.any() else 0.0,
            "nan_left": bool(np.isnan(og).any() or np.isnan(lg).any()),
            "inf_pattern_equal": bool(np.array_equal(np.isfinite(lg), fin)),
            "tol_o": 2e-2, "tol_lse": 1e-3,
        }
        p = out["parity"]
        p["ok"] = bool(p["max_abs_o"] <= 2e-2 and p["max_abs_lse"] <= 1e-3 and not p["nan_left"] and p["inf_pattern_equal"])
    return out


def cpu_baseline_gemm(a, b, target_seconds, c_gpu=None):
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
    idx = entries(n)
    t0 = time.perf_counter()
    ref = oracle.gemm_tn_entries(a, b, idx)
    dt = time.perf_counter() - t0
    out = {"value": 2.0 * K * n / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "%d of %d entries of C (%dx%dx%d), evenly spread, %.1f s; 2*K flops per entry" % (n, M * N, M, N, K, dt),
           "seconds": dt}
    if c_gpu is not None:
        got = c_gpu[idx[:, 0], idx[:, 1]].double().numpy()
        tol = np.abs(ref) * 2.0 ** -8 + 1e-3 * np.sqrt(K)
        out["parity"] = {"entries": int(n), "max_abs_c": float(np.abs(got - ref).max()),
                         "max_err_over_tol": float((np.abs(got - ref) / tol).max()),
                         "tol": "2^-8*|C| + 1e-3*sqrt(K)", "ok": bool((np.abs(got - ref) <= tol).all())}
    return out


# ----------------------------------------------------------------- reference arm
def run_reference(args):
    """The reference arm: the fp64 CPU oracle, as it stands, on the host cores.  Rank 0 alone works."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    from paper_2604_18616_b200 import inputs
    steps, warm = max(1, args.steps), max(0, args.warmup)
    per_step = max(0.5, min(args.cpu_seconds, 150.0 / (steps + warm)))
    is_gemm = args.workload.startswith("gemm_n")
    is_moe = args.workload.startswith("moe_t")
    if is_moe:
        mw = inputs.MOE_WORKLOADS[args.workload]
        margs = inputs.make_moe_inputs(mw)
        sample = lambda: cpu_baseline_moe(mw, margs, per_step)
        config = {"workload": mw.name, "T": mw.T, "C": mw.C, "F": mw.F, "E": mw.E, "K": mw.K}
    elif is_gemm:
        n = gemm_size(args.workload)
        a, b = inputs.make_gemm_inputs(n, n, n, seed=20)
        sample = lambda: cpu_baseline_gemm(a, b, per_step)
        config = {"workload": args.workload, "M": n, "N": n, "K": n}
    else:
        w = inputs.get(args.workload)
        q, k, v = inputs.make_inputs(w)
        sample = lambda: cpu_baseline_attention(w, q, k, v, per_step)
        config = workload_config(w)
    for _ in range(warm):
        sample()
    recs = [sample() for _ in range(steps)]
    value = sum(r["value"] for r in recs) / len(recs)
    total = sum(r["seconds"] for r in recs)
    print(json.dumps({
        "impl": "reference", "metric": GEMM_METRIC if is_gemm else MOE_METRIC if is_moe else METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": 1e3 * total / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": recs[-1]["cores"], "kind": "oracle",
                         "sample": "each step: " + recs[-1]["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))
    return 0


# ------------------------------------------------------------------------ GPU legs
class Ctx:
    """What every GPU leg needs: device, stream, ranks, peaks, clock sampler."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        self.torch, self.dist, self.args = torch, dist, args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.peak, self.peak_sustained, self.hbm_gbs, self.peak_kind = measured_peaks()

    def init_gpu(self):
        torch = self.torch
        from paper_2604_18616_b200 import binding
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the attention path has no CPU fallback")
        binding.lib()   # raises if the CUDA library is not built
        binding.select_kernel(self.args.kernel)
        torch.cuda.set_device(self.local_rank)
        self.dev = torch.device("cuda", self.local_rank)
        if self.world > 1:
            self.dist.init_process_group("nccl", device_id=self.dev)
        self.stream = torch.cuda.current_stream()
        pr = torch.cuda.get_device_properties(self.local_rank)
        try:
            bus = "%08x:%02x:%02x.0" % (pr.pci_domain_id, pr.pci_bus_id, pr.pci_device_id)
        except AttributeError:
            bus = None
        self.clocks = ClockSampler(self.local_rank, bus)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, values):
        t = self.torch.tensor(values, dtype=self.torch.float64, device=self.dev)
        if self.world > 1:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return t.tolist()

    def check_status(self, where):
        from paper_2604_18616_b200 import binding
        st, raw = binding.device_status()
        if st != binding.AVE_OK:
            raise RuntimeError("device status %d (raw %#x) after %s" % (st, raw, where))


def attention_ceilings(w):
    """Upper bounds of the kernel's own structure at the maximum SM clock, from the measured unit rates: the
    tensor pipe (QK^T and PV of a 128 x 128 step) and the exponential unit (128 x 128 results per step)."""
    clk_hz = 1965e6
    qk = (w.D / 16.0) * MMA_CLK_N128 if w.D > 64 else (64 / 16.0) * MMA_CLK_N128
    pv = 8 * (MMA_CLK_N128 * (w.D / 128.0) if w.D > 64 else MMA_CLK_N64)
    flop_step = 4.0 * 128 * 128 * w.D
    tensor = flop_step / (qk + pv) * clk_hz * N_SMS / 1e12
    exp_all = flop_step / (128 * 128 / EX2_PER_CLK) * clk_hz * N_SMS / 1e12
    return {"tensor_pipe_tflops": tensor, "exp_unit_tflops": exp_all,
            "exp_unit_with_quarter_on_fma_pipe_tflops": exp_all / 0.75,
            "note": "executed (tile-granular) work at 1965 MHz; causal workloads execute slightly more than the counted half"}


def attention_leg(ctx, w, steps, warmup, headline):
    """Time K launches of one attention workload, then check a poisoned launch against oracle rows."""
    torch = ctx.torch
    from paper_2604_18616_b200 import binding, inputs, shard
    args = ctx.args
    # N > 1, weak: an independent batch of the same shape per rank; strong: this rank's (batch, KV head) units
    wr = inputs.small_variant(w, seed=w.seed + 1000 * ctx.rank) if (ctx.rank > 0 and args.scaling == "weak") else w
    q, k, v = inputs.make_inputs(wr)
    if ctx.world > 1 and args.scaling == "strong":
        qs, ks, vs, (lo, hi) = shard.shard_qkv(q, k, v, ctx.world, ctx.rank)
        q, k, v = qs.contiguous(), ks.contiguous(), vs.contiguous()
        wr = inputs.small_variant(w, B=hi - lo, H=w.G, Hkv=1)
    Bq, Hq = q.shape[0], q.shape[1]
    n_sets = rotation_sets(inputs.min_hbm_bytes(wr))
    sets = []
    for _ in range(n_sets):
        sets.append((q.to(ctx.dev), k.to(ctx.dev), v.to(ctx.dev), torch.empty(q.shape, dtype=torch.bfloat16, device=ctx.dev),
                     torch.empty((Bq, Hq, wr.Sq), dtype=torch.float32, device=ctx.dev)))
    flops = inputs.attn_flops(wr)

    def step(i):
        qd, kd, vd, o, lse = sets[i % n_sets]
        binding.ave_attn_fwd(qd, kd, vd, o, lse, causal=wr.causal, scale=wr.scale, stream=ctx.stream)

    for i in range(max(warmup, 3)):
        step(i)
    ctx.barrier()
    n0 = binding.launch_count()
    ms = timed_launches(torch, ctx.stream, step, steps, ctx.clocks, ctx.barrier)
    launches = binding.launch_count() - n0
    clocks = ctx.clocks.summary()
    ctx.check_status("the timed region of " + w.name)
    rec = {"workload": w.name, "kind": "attention", "config": workload_config(wr), "steps": steps,
           "us": 1e3 * ms / steps, "tflops": flops / (ms / steps * 1e-3) / 1e12, "gpu_launches": int(launches),
           "clocks": clocks, "input_sets": n_sets, "_ms": ms, "_flops": flops}
    rec["frac"] = rec["tflops"] / ctx.peak
    if w.D <= 64:
        rec["ceilings"] = attention_ceilings(w)

    # ---- a launch into NaN-poisoned outputs, outside the timed region, for the oracle check
    qd, kd, vd, o, lse = sets[0]
    o.fill_(float("nan"))
    lse.fill_(float("nan"))
    step(0)
    ctx.check_status("the checked launch of " + w.name)
    rec["_q"], rec["_k"], rec["_v"], rec["_o"], rec["_lse"], rec["_w"] = q, k, v, o.cpu(), lse.cpu(), wr
    rec["input_sha256"] = {"q": inputs.tensor_sha256(q)[:16], "k": inputs.tensor_sha256(k)[:16],
                           "v": inputs.tensor_sha256(v)[:16]}

    if headline:
        # the rate the same loop settles at under the power cap, with its own clock record
        if args.sustain_seconds > 0 and ctx.world == 1:
            n_long = int(max(steps, args.sustain_seconds / max(1e-6, ms / steps * 1e-3)))
            ms_long = timed_launches(torch, ctx.stream, step, n_long, ctx.clocks)
            cl = ctx.clocks.summary()
            tf = flops / (ms_long / n_long * 1e-3) / 1e12
            capped = "sw_power_cap" in cl["reasons"] and ms_long >= 1000.0
            rec["sustained"] = {"launches": n_long, "seconds": ms_long * 1e-3, "tflops": tf, "frac": tf / ctx.peak,
                                "clocks": cl, "peak_sustained": ctx.peak_sustained,
                                "frac_of_sustained": (tf / ctx.peak_sustained) if (capped and ctx.peak_sustained) else None}
            ctx.check_status("the sustained loop")
        # ---- end to end: pinned host buffers in, host buffers out, copies inside the timed region
        e2e_steps = max(1, min(args.e2e_steps, steps))
        qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
        oh = torch.empty_like(q).pin_memory()
        lh = torch.empty((Bq, Hq, wr.Sq), dtype=torch.float32).pin_memory()
        ws = torch.empty(binding.host_workspace_bytes(Bq, Hq, wr.Hkv, wr.Sq, wr.Sk, wr.D), dtype=torch.uint8, device=ctx.dev)

        def e2e_step(i):
            binding.ave_attn_fwd_host(qh, kh, vh, oh, lh, ws, causal=wr.causal, scale=wr.scale, stream=ctx.stream)

        for i in range(3):
            e2e_step(i)
        ctx.barrier()
        e2e_ms = timed_launches(torch, ctx.stream, e2e_step, e2e_steps, ctx.clocks, ctx.barrier)
        ctx.check_status("the end-to-end loop")
        rec["_e2e"] = {"ms": e2e_ms, "steps": e2e_steps, "h2d": (q.numel() + k.numel() + v.numel()) * 2,
                       "d2h": oh.numel() * 2 + lh.numel() * 4,
                       "result_equal_to_device_path": bool(torch.equal(oh, rec["_o"]) and torch.equal(lh, rec["_lse"]))}
    del sets
    torch.cuda.empty_cache()
    return rec


def decode_leg(ctx, w, steps, warmup):
    """Split-KV decode: few query rows against many keys; HBM roofline on the unique K+V (+Q, O) bytes."""
    torch = ctx.torch
    from paper_2604_18616_b200 import binding, inputs
    q, k, v = inputs.make_inputs(w)
    n_splits = binding.splitkv_default_splits(w.B, w.H, w.Hkv, w.Sq, w.Sk, w.D)
    bytes_alg = inputs.min_hbm_bytes(w)
    n_sets = rotation_sets(bytes_alg)
    ws = torch.empty(max(256, binding.splitkv_workspace_bytes(w.B, w.H, w.Sq, w.D, n_splits)), dtype=torch.uint8, device=ctx.dev)
    sets = [(q.to(ctx.dev), k.to(ctx.dev), v.to(ctx.dev), torch.empty(q.shape, dtype=torch.bfloat16, device=ctx.dev),
             torch.empty((w.B, w.H, w.Sq), dtype=torch.float32, device=ctx.dev)) for _ in range(n_sets)]

    def step(i):
        qd, kd, vd, o, lse = sets[i % n_sets]
        binding.ave_attn_fwd_splitkv(qd, kd, vd, n_splits, ws, o, lse, causal=w.causal, scale=w.scale, stream=ctx.stream)

    for i in range(max(warmup, 3)):
        step(i)
    ctx.barrier()
    n0 = binding.launch_count()
    ms = timed_launches(torch, ctx.stream, step, steps, ctx.clocks, ctx.barrier)
    launches = binding.launch_count() - n0
    clocks = ctx.clocks.summary()
    ctx.check_status("the timed region of " + w.name)
    us = 1e3 * ms / steps
    gbs = bytes_alg / (us * 1e-6) / 1e9
    rec = {"workload": w.name, "kind": "splitkv_decode", "config": dict(workload_config(w), n_splits=n_splits),
           "steps": steps, "us": us, "tflops": inputs.attn_flops(w) / (us * 1e-6) / 1e12, "gpu_launches": int(launches),
           "clocks": clocks, "input_sets": n_sets,
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": ctx.hbm_gbs, "unit": "GB/s", "frac": gbs / ctx.hbm_gbs,
                        "algorithmic_hbm_bytes": bytes_alg, "kernels_per_step": 2},
           "_ms": ms, "_flops": inputs.attn_flops(w)}
    rec["frac"] = rec["roofline"]["frac"]
    qd, kd, vd, o, lse = sets[0]
    o.fill_(float("nan"))
    lse.fill_(float("nan"))
    step(0)
    ctx.check_status("the checked launch of " + w.name)
    rec["_q"], rec["_k"], rec["_v"], rec["_o"], rec["_lse"], rec["_w"] = q, k, v, o.cpu(), lse.cpu(), w
    rec["input_sha256"] = {"q": inputs.tensor_sha256(q)[:16], "k": inputs.tensor_sha256(k)[:16],
                           "v": inputs.tensor_sha256(v)[:16]}
    del sets, ws
    torch.cuda.empty_cache()
    return rec


def gemm_size(name):
    """'gemm_n8192' -> 8192 (square product, the paper's Section 9 GEMM workload)."""
    n = int(name[len("gemm_n"):])
    if n <= 0 or n % 8:
        raise ValueError("gemm_n<size>: size must be a positive multiple of 8")
    return n


def gemm_leg(ctx, name, steps, warmup, headline):
    torch = ctx.torch
    from paper_2604_18616_b200 import binding, inputs
    n = gemm_size(name)
    a, b = inputs.make_gemm_inputs(n, n, n, seed=20 + 1000 * ctx.rank)   # an independent product per rank
    n_sets = rotation_sets(3 * n * n * 2)
    sets = [(a.to(ctx.dev), b.to(ctx.dev), torch.empty((n, n), dtype=torch.bfloat16, device=ctx.dev)) for _ in range(n_sets)]
    flops = 2.0 * n * n * n

    def step(i):
        ad, bd, c = sets[i % n_sets]
        binding.ave_gemm_bf16_tn(ad, bd, c, stream=ctx.stream)

    for i in range(max(warmup, 3)):
        step(i)
    ctx.barrier()
    n0 = binding.launch_count()
    ms = timed_launches(torch, ctx.stream, step, steps, ctx.clocks, ctx.barrier)
    launches = binding.launch_count() - n0
    clocks = ctx.clocks.summary()
    ctx.check_status("the timed region of " + name)
    rec = {"workload": name, "kind": "gemm", "config": {"workload": name, "M": n, "N": n, "K": n,
                                                        "layout": "A [M,K], B [N,K], C [M,N] row-major"},
           "steps": steps, "us": 1e3 * ms / steps, "tflops": flops / (ms / steps * 1e-3) / 1e12,
           "gpu_launches": int(launches), "clocks": clocks, "input_sets": n_sets, "_ms": ms, "_flops": flops}
    rec["frac"] = rec["tflops"] / ctx.peak
    # the vendor library on the same operands, same process, same number of launches: context, not the path
    ad, bd, c = sets[0]
    out = torch.empty_like(c)
    for _ in range(3):
        torch.matmul(ad, bd.t(), out=out)
    torch.cuda.synchronize()
    ms_lib = timed_launches(torch, ctx.stream, lambda i: torch.matmul(sets[i % n_sets][0], sets[i % n_sets][1].t(), out=out),
                            steps, ctx.clocks)
    rec["torch_matmul_tflops"] = flops / (ms_lib / steps * 1e-3) / 1e12
    c.fill_(float("nan"))
    step(0)
    ctx.check_status("the checked launch of " + name)
    rec["_a"], rec["_b"], rec["_c"] = a, b, c.cpu()
    rec["input_sha256"] = {"a": inputs.tensor_sha256(a)[:16], "b": inputs.tensor_sha256(b)[:16]}
    if headline:
        e2e_steps = max(1, min(ctx.args.e2e_steps, steps))
        ah, bh = a.pin_memory(), b.pin_memory()
        ch = torch.empty((n, n), dtype=torch.bfloat16).pin_memory()

        def e2e_step(i):
            ad.copy_(ah, non_blocking=True)
            bd.copy_(bh, non_blocking=True)
            binding.ave_gemm_bf16_tn(ad, bd, c, stream=ctx.stream)
            ch.copy_(c, non_blocking=True)

        for i in range(3):
            e2e_step(i)
        ctx.barrier()
        e2e_ms = timed_launches(torch, ctx.stream, e2e_step, e2e_steps, ctx.clocks, ctx.barrier)
        rec["_e2e"] = {"ms": e2e_ms, "steps": e2e_steps, "h2d": 2 * n * n * 2, "d2h": n * n * 2,
                       "result_equal_to_device_path": bool(torch.equal(ch, rec["_c"]))}
    del sets
    torch.cuda.empty_cache()
    return rec


def cpu_baseline_moe(w, args, target_seconds, y_gpu=None):
    """The oracle on a bounded sample of tokens (each costs K * 3 * C * F multiply-adds in fp64)."""
    import numpy as np
    import oracle
    from paper_2604_18616_b200 import inputs
    a = [t.numpy() for t in args]
    cores = oracle.threads()
    probe = list(range(min(w.T, max(1, cores))))
    t0 = time.perf_counter()
    oracle.moe_rows(*a, tokens=probe)
    t_probe = time.perf_counter() - t0
    n = int(min(w.T, max(len(probe), len(probe) * target_seconds / max(t_probe, 1e-6))))
    tok = np.unique(np.linspace(0, w.T - 1, n).astype(np.int64))
    t0 = time.perf_counter()
    y_ref = oracle.moe_rows(*a, tokens=tok)
    dt = time.perf_counter() - t0
    out = {"value": inputs.moe_flops(w) * len(tok) / w.T / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "%d of %d tokens of %s, evenly spread, %.1f s" % (len(tok), w.T, w.name, dt), "seconds": dt}
    if y_gpu is not None:
        got = y_gpu[tok].double().numpy()
        rms = float(np.sqrt(np.mean(y_ref ** 2))) + 1e-30
        err = np.abs(got - y_ref)
        tight = 2.0 ** -7 * np.abs(y_ref) + 2e-3 * rms
        one_step = float(a[7].max()) * 448.0 * float(a[5].max())
        out["parity"] = {"tokens": int(len(tok)), "max_abs_y": float(err.max()), "rms_y": rms,
                         "frac_outside_tight": float(np.mean(err > tight)), "nan_left": bool(np.isnan(got).any()),
                         "tol": "all within 2^-7|y| + one E4M3 step of an intermediate; 99.8 % within 2^-7|y| + 2e-3 rms",
                         "ok": bool(np.mean(err > tight) <= 2e-3 and np.all(err <= 2.0 ** -7 * np.abs(y_ref) + one_step)
                                    and not np.isnan(got).any())}
    return out


def moe_leg(ctx, name, steps, warmup, headline):
    torch = ctx.torch
    from paper_2604_18616_b200 import binding, inputs
    w = inputs.MOE_WORKLOADS[name]
    args = inputs.make_moe_inputs(w)
    d = [t.to(ctx.dev) for t in args]
    y = torch.empty((w.T, w.C), dtype=torch.bfloat16, device=ctx.dev)
    ws = torch.empty(binding.moe_workspace_bytes(w.T, w.C, w.F, w.E, w.K), dtype=torch.uint8, device=ctx.dev)
    flops = inputs.moe_flops(w)

    def step(i):
        binding.ave_moe_fused_fwd(*d, y=y, workspace=ws, stream=ctx.stream)

    for i in range(max(warmup, 3)):
        step(i)
    ctx.barrier()
    n0 = binding.launch_count()
    ms = timed_launches(torch, ctx.stream, step, steps, ctx.clocks, ctx.barrier)
    launches = binding.launch_count() - n0
    clocks = ctx.clocks.summary()
    ctx.check_status("the timed region of " + name)
    peak8 = ctx.peak * FP8_OVER_BF16
    weight_bytes = w.E * 3 * w.C * w.F
    rec = {"workload": name, "kind": "moe", "config": {"workload": name, "T": w.T, "C": w.C, "F": w.F, "E": w.E, "K": w.K},
           "steps": steps, "us": 1e3 * ms / steps, "tflops": flops / (ms / steps * 1e-3) / 1e12,
           "gpu_launches": int(launches), "clocks": clocks, "input_sets": 1,
           "roofline": {"bound": "tensor", "achieved": flops / (ms / steps * 1e-3) / 1e12, "peak": peak8, "unit": UNIT,
                        "peak_kind": "measured bf16 matmul rate x the nominal fp8/bf16 ratio of 2",
                        "algorithmic_hbm_bytes": weight_bytes + w.T * w.C * 3, "kernels_per_step": 7},
           "_ms": ms, "_flops": flops}
    rec["roofline"]["frac"] = rec["roofline"]["achieved"] / peak8
    rec["frac"] = rec["roofline"]["frac"]
    y.fill_(float("nan"))
    step(0)
    ctx.check_status("the checked launch of " + name)
    rec["_moe"], rec["_args"], rec["_y"] = w, args, y.cpu()
    rec["input_sha256"] = {"xq": inputs.tensor_sha256(args[0])[:16], "ids": inputs.tensor_sha256(args[6])[:16]}
    if headline:
        e2e_steps = max(1, min(ctx.args.e2e_steps, steps))
        # the activations and the routing come from the host every step; the weights stay resident (a layer's weights
        # do not change between calls)
        hx, hs, hi, hw = (args[i].pin_memory() for i in (0, 1, 6, 7))
        hy = torch.empty((w.T, w.C), dtype=torch.bfloat16).pin_memory()

        def e2e_step(i):
            d[0].copy_(hx, non_blocking=True)
            d[1].copy_(hs, non_blocking=True)
            d[6].copy_(hi, non_blocking=True)
            d[7].copy_(hw, non_blocking=True)
            binding.ave_moe_fused_fwd(*d, y=y, workspace=ws, stream=ctx.stream)
            hy.copy_(y, non_blocking=True)

        for i in range(3):
            e2e_step(i)
        ctx.barrier()
        e2e_ms = timed_launches(torch, ctx.stream, e2e_step, e2e_steps, ctx.clocks, ctx.barrier)
        rec["_e2e"] = {"ms": e2e_ms, "steps": e2e_steps, "h2d": sum(args[i].numel() * args[i].element_size() for i in (0, 1, 6, 7)),
                       "d2h": hy.numel() * 2, "result_equal_to_device_path": bool(torch.equal(hy, rec["_y"]))}
    del d, ws
    torch.cuda.empty_cache()
    return rec


def finish_record(rec, cpu_seconds, want_oracle):
    """Run the CPU-baseline leg of a record (oracle timing + comparison with the GPU rows) and drop the tensors."""
    if want_oracle:
        if rec["kind"] == "gemm":
            rec["cpu_baseline"] = cpu_baseline_gemm(rec["_a"], rec["_b"], cpu_seconds, rec["_c"])
        elif rec["kind"] == "moe":
            rec["cpu_baseline"] = cpu_baseline_moe(rec["_moe"], rec["_args"], cpu_seconds, rec["_y"])
        else:
            rec["cpu_baseline"] = cpu_baseline_attention(rec["_w"], rec["_q"], rec["_k"], rec["_v"], cpu_seconds,
                                                         rec["_o"], rec["_lse"], spread=False)
        par = rec["cpu_baseline"].pop("parity")
        rec["parity"] = par
    for key in [k for k in rec if k.startswith("_") and k not in ("_ms", "_flops", "_e2e")]:
        del rec[key]
    return rec


def run_leg(ctx, name, steps, warmup, headline=False):
    from paper_2604_18616_b200 import inputs
    if name.startswith("gemm_n"):
        return gemm_leg(ctx, name, steps, warmup, headline)
    if name.startswith("moe_t"):
        return moe_leg(ctx, name, steps, warmup, headline)
    w = inputs.get(name)
    if name.startswith("decode_"):
        return decode_leg(ctx, w, steps, warmup)
    return attention_leg(ctx, w, steps, warmup, headline)


def run_ours(args):
    ctx = Ctx(args)
    ctx.init_gpu()
    torch = ctx.torch
    from paper_2604_18616_b200 import inputs
    steps, warmup = max(1, args.steps), max(args.warmup, 3)
    head = run_leg(ctx, args.workload, steps, warmup, headline=True)
    e2e = head.get("_e2e")
    ms_max, e2e_ms_max = ctx.max_over_ranks([head["_ms"], e2e["ms"] if e2e else 0.0])
    want_oracle = not args.no_cpu_baseline and ctx.world == 1 and ctx.rank == 0
    if ctx.rank == 0:
        flops = head["_flops"]
        ms_per_step = ms_max / steps
        is_gemm = head["kind"] == "gemm"
        is_moe = head["kind"] == "moe"
        finish_record(head, args.cpu_seconds, want_oracle)
        kernel_tf = head["tflops"]
        if head["kind"] == "splitkv_decode":
            roofline = dict(head["roofline"], traffic=NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload), peak_kind=ctx.peak_kind)
        elif is_moe:
            roofline = dict(head["roofline"], traffic=NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload))
        else:
            w = None if is_gemm else inputs.get(args.workload)
            roofline = {"bound": "tensor", "achieved": kernel_tf, "peak": ctx.peak, "unit": UNIT,
                        "frac": kernel_tf / ctx.peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload),
                        "traffic_unit": "bytes per launch (ncu dram read+write)",
                        "algorithmic_hbm_bytes": (3 * gemm_size(args.workload) ** 2 * 2) if is_gemm else inputs.min_hbm_bytes(w),
                        "peak_kind": ctx.peak_kind + "; frac is of the burst rate, the stricter of the two measured",
                        "frac_of_nominal_2250": kernel_tf / NOMINAL_BF16_TFLOPS,
                        "flops_per_launch": flops, "kernel_us": head["us"]}
        cfg = dict(head["config"])
        cfg["parallelism"] = "dp%d (%s)" % (ctx.world, "independent batches, no collective" if args.scaling == "weak"
                                            else "one batch sharded over (batch, KV head) units, no collective")
        cfg["l2"] = ("inputs+outputs of a step exceed the 126 MB L2; no explicit flush" if head["input_sets"] == 1 else
                     "launches rotate over %d input/output sets so that a launch does not find its operands in L2" % head["input_sets"])
        line = {
            "metric": GEMM_METRIC if is_gemm else MOE_METRIC if is_moe else METRIC,
            "value": ctx.world * flops / (ms_per_step * 1e-3) / 1e12,
            "unit": UNIT, "n_gpus": ctx.world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None, "dtype": "fp8_e4m3" if is_moe else "bf16",
            "data": "synthetic", "config": cfg, "clocks": head["clocks"], "gpu_launches": head["gpu_launches"],
            "roofline": roofline, "input_sha256": head["input_sha256"],
        }
        if e2e:
            line["e2e"] = {"value": ctx.world * flops / (e2e_ms_max / e2e["steps"] * 1e-3) / 1e12, "unit": UNIT,
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"],
                           "result_equal_to_device_path": e2e["result_equal_to_device_path"]}
        for key in ("sustained", "ceilings", "parity", "cpu_baseline", "torch_matmul_tflops"):
            if key in head:
                line[key] = head[key]
        # ---- the other workloads, one record each (1 GPU only: N > 1 runs hold all N GPUs meanwhile)
        legs = [] if args.legs == "none" or ctx.world > 1 else (
            PER_WORKLOAD_DEFAULT if args.legs == "all" else [s for s in args.legs.split(",") if s])
        per = []
        for name in legs:
            if name == args.workload:
                r = {k: head[k] for k in ("workload", "kind", "config", "steps", "us", "tflops", "frac", "clocks",
                                          "input_sha256", "parity") if k in head}
                per.append(r)
                continue
            try:
                r = run_leg(ctx, name, steps, warmup)
                finish_record(r, args.leg_cpu_seconds, want_oracle)
                for key in ("_ms", "_flops", "_e2e"):
                    r.pop(key, None)
                if "cpu_baseline" in r:
                    r["cpu_baseline"] = {k: r["cpu_baseline"][k] for k in ("value", "cores", "sample")}
                per.append(r)
            except KeyError:
                per.append({"workload": name, "error": "unknown workload"})
        if per:
            line["per_workload"] = per
            line["parity_all_ok"] = all(r.get("parity", {}).get("ok", False) for r in per if "error" not in r) if want_oracle else None
        print(json.dumps(line))
    if ctx.world > 1:
        ctx.dist.barrier()
        ctx.dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------- rank start-up
def rank_plan(args):
    """Every rank reports what it would run; rank 0 prints the list.  Uses NCCL on GPUs, gloo on a CPU machine."""
    import torch
    import torch.distributed as dist
    from paper_2604_18616_b200 import inputs, shard
    world, rank = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    gpu = torch.cuda.is_available()
    if world > 1:
        if gpu:
            torch.cuda.set_device(local_rank)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group("gloo")
    w = inputs.get(args.workload)
    mine = {"rank": rank, "local_rank": local_rank, "device": ("cuda:%d" % local_rank) if gpu else "cpu"}
    if args.scaling == "weak":
        mine.update(seed=w.seed + 1000 * rank, units=[0, w.B * w.Hkv])
    else:
        mine.update(seed=w.seed, units=list(shard.unit_range(w.B * w.Hkv, world, rank)))
    plan = [mine]
    if world > 1:
        plan = [None] * world
        dist.all_gather_object(plan, mine)
        # the timing reduction of the real run: max over ranks
        t = torch.tensor([float(rank + 1)], dtype=torch.float64, device="cuda" if gpu else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == world
    if rank == 0:
        print(json.dumps({"plan": plan, "n_gpus": world, "scaling": args.scaling, "workload": w.name,
                          "backend": "nccl" if gpu else "gloo"}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def main(argv=None):
    args = parse_args(argv)
    # `--gpus N` without a torchrun environment: start the N ranks here, one process per GPU
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.plan_only):
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + \
            (list(argv) if argv is not None else sys.argv[1:])
        return subprocess.run(cmd).returncode
    if args.plan_only:
        return rank_plan(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
