"""Host-side pieces of bench.py that need no GPU: the two arms describe the workload identically, the
reference arm honours --steps/--warmup, input rotation and clock sampling behave on a box without NVML."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2604_18616_b200 import inputs  # noqa: E402


def test_reference_arm_runs_the_oracle_with_the_requested_steps():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1_tiny",
                        "--steps", "3", "--warmup", "1", "--cpu-seconds", "0.5"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 3 and line["warmup"] == 1
    assert line["metric"] == bench.METRIC and line["unit"] == "TFLOP/s" and line["higher_is_better"] is True
    assert line["config"] == bench.workload_config(inputs.get("c1_tiny"))       # the GPU arm's config object
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["value"] > 0 and line["gpu_launches"] == 0


def test_default_headline_is_the_largest_prefill_configuration():
    args = bench.parse_args([])
    assert args.workload == "c4_long_context" and args.gpus == 1 and args.warmup >= 3
    for name in bench.PER_WORKLOAD_DEFAULT:
        assert name.startswith("gemm_n") or name in inputs.WORKLOADS or name in inputs.MOE_WORKLOADS
    for n in ("c1_tiny", "c2_mha_prefill", "c3_gqa_prefill", "c4_long_context", "c5_wide_noncausal",
              "paper_gqa_n1024", "paper_gqa_n16384"):
        assert n in bench.PER_WORKLOAD_DEFAULT


def test_rotation_keeps_consecutive_launches_out_of_l2():
    assert bench.rotation_sets(inputs.min_hbm_bytes(inputs.get("c4_long_context"))) == 1      # 322 MiB: beyond L2 anyway
    n = bench.rotation_sets(inputs.min_hbm_bytes(inputs.get("paper_gqa_n1024")))
    assert n >= 2 and n * inputs.min_hbm_bytes(inputs.get("paper_gqa_n1024")) >= 2 * bench.L2_BYTES
    assert bench.rotation_sets(130_000) == 32                                                 # capped for tiny problems


def test_clock_sampler_reports_instead_of_failing_without_nvml():
    c = bench.ClockSampler(0)
    with c:
        c.sample()
    s = c.summary()
    assert set(s) >= {"sm_mhz", "sm_max_mhz", "reasons", "samples"}


def test_ceilings_of_the_narrow_head_kernel():
    c = bench.attention_ceilings(inputs.get("c5_wide_noncausal"))
    # at D = 64 the exponential unit, not the tensor pipe, is the lower ceiling
    assert c["exp_unit_tflops"] < c["tensor_pipe_tflops"]
    assert 1100 < c["exp_unit_tflops"] < 1300 and 1800 < c["tensor_pipe_tflops"] < 2100


def test_timeline_decodes_the_stamp_array():
    """The profiling aid's host side: stamps [role][iteration][slot] -> time-ordered events; iterations 32.. belong
    to the second traced tile, 28 / 30 are the producer's and the epilogue's per-tile stamps."""
    from paper_2604_18616_b200 import timeline as t
    st = [0] * (t.ROLES * t.ITERS * t.SLOTS)
    at = lambda role, it, sl: (role * t.ITERS + it) * t.SLOTS + sl
    st[at(3, 2, 7)] = 800
    st[at(0, 3, 0)] = 900
    st[at(1, 3, 1)] = 1000
    st[at(2, 62, 2)] = 2000
    st[at(3, 28, 1)] = 1500
    ev = t.events(st)
    assert [e[0] for e in ev] == [0, 100, 200, 700, 1200]
    assert ev[0][1] == "MMA" and "tile number 2" in ev[0][2]
    assert ev[2] == (200, "SM0", "T0 j=3 S ready")
    assert ev[3] == (700, "LD ", "T0 Q0 issue")
    assert ev[4] == (1200, "SM1", "T1 epilogue done")
    assert t.events([0] * len(st)) == []


def test_timeline_span_summary():
    """Per-CTA (first ns, last ns, tiles) triples -> kernel span, how ragged the start and the end are, average
    residency; CTAs whose index a running CTA took over have no start and are left out."""
    from paper_2604_18616_b200 import timeline as t
    txt = t.span_summary([(1000, 9000, 3), (1500, 8000, 2), (0, 0, 0), (2000, 9500, 4)], sms=4)
    assert "CTAs that ran: 3 of 4" in txt and "8.50 us" in txt
    assert "max 1.00" in txt and "max 1.50" in txt            # latest start, earliest end
    assert "2.6 CTAs resident" in txt                         # (8000 + 6500 + 7500) / 8500
    assert "min 2, max 4, total 9" in txt
    assert t.span_summary([(0, 0, 0)] * 5) == "no CTA ran"
