"""Role timeline of one CTA of the attention kernel (a profiling aid).

``python -m paper_2604_18616_b200.timeline <workload> [--cta N] [--tile K]`` builds a trace variant
of the library (``-DAVE_TRACE=<cta> -DAVE_TRACE_TILE=<k>``, written beside the normal one as
``libave_attn_trace.so``), runs the named workload on cuda:0 and prints, in time order, the SM-clock
stamps that the producer, MMA and softmax warps of that CTA took during its k-th and (k+1)-th work
tiles: where a key step's time goes, and what a tile boundary costs.  The normal library carries no
trace code.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess
import sys

from . import build

TRACE_LIB = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libave_attn_trace.so")
ROLES, ITERS, SLOTS = 4, 64, 8          # dimensions of the device-side stamp array
NAMES = {0: "MMA", 1: "SM0", 2: "SM1", 3: "LD "}
LABELS = {0: ["round start", "P0 taken", "PV0+QK0 issued", "P1 taken", "PV1+QK1 issued"],
          1: ["wait S", "S ready", "S in registers", "row max done", "exp done", "P handed over"],
          2: ["wait S", "S ready", "S in registers", "row max done", "exp done", "P handed over"],
          3: ["K issue", "V issue"]}


def build_trace_library(cta: int, tile: int) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = [f for f in build.NVCC_FLAGS if f not in ("-Xptxas", "-v")]
    cmd = [nvcc] + flags + ["-DAVE_TRACE=%d" % cta, "-DAVE_TRACE_TILE=%d" % tile, "-o", TRACE_LIB,
                            os.path.join(build.CSRC, "ave_attn.cu")]
    subprocess.run(cmd, check=True)
    return TRACE_LIB


def events(stamps):
    """[(clock, role name, text)] from the [ROLES][ITERS][SLOTS] stamp array (0 = not taken)."""
    taken = [x for x in stamps if x > 0]
    if not taken:
        return []
    base = min(taken)
    out = []
    for role in range(ROLES):
        for it in range(ITERS):
            for sl in range(SLOTS):
                x = stamps[(role * ITERS + it) * SLOTS + sl]
                if x <= 0:
                    continue
                tile, j = divmod(it, 32)
                if role == 3 and sl == 7:
                    text = "the CTA's tile number %d starts" % it
                    who = "MMA"
                elif j == 28:
                    lab = ["tile loop start", "Q0 issue", "Q1 issue", "all loads issued", "next tile known"]
                    text = "T%d %s" % (tile, lab[sl] if sl < len(lab) else "stamp %d" % sl)
                    who = NAMES[role]
                elif j == 30:
                    lab = ["epilogue: wait for O", "epilogue: O ready", "epilogue done", "next tile known"]
                    text = "T%d %s" % (tile, lab[sl] if sl < len(lab) else "stamp %d" % sl)
                    who = NAMES[role]
                else:
                    lab = LABELS[role]
                    text = "T%d j=%d %s" % (tile, j, lab[sl] if sl < len(lab) else "stamp %d" % sl)
                    who = NAMES[role]
                out.append((x - base, who, text))
    out.sort()
    return out


def span_summary(spans, sms=148):
    """Text summary of per-CTA (first ns, last ns, tiles) triples of one launch; CTAs that never ran
    (their index was taken over by a running CTA) have a zero start."""
    ran = [(a, b, t) for a, b, t in spans if a > 0 and b >= a]
    if not ran:
        return "no CTA ran"
    t0 = min(a for a, _, _ in ran)
    t1 = max(b for _, b, _ in ran)
    starts = sorted(a - t0 for a, _, _ in ran)
    ends = sorted(t1 - b for _, b, _ in ran)
    busy = sum(b - a for a, b, _ in ran)
    mid = len(ran) // 2
    lines = ["CTAs that ran: %d of %d; kernel span (first start to last end): %.2f us" % (len(ran), len(spans), (t1 - t0) / 1e3),
             "start after the first CTA's start, us: median %.2f, 90%% %.2f, max %.2f" % (
                 starts[mid] / 1e3, starts[int(0.9 * (len(ran) - 1))] / 1e3, starts[-1] / 1e3),
             "end before the last CTA's end, us: median %.2f, 90%% %.2f, max %.2f" % (
                 ends[mid] / 1e3, ends[int(0.9 * (len(ran) - 1))] / 1e3, ends[-1] / 1e3),
             "CTA life summed / kernel span: %.1f CTAs resident on average (the GPU has %d SMs)" % (busy / max(1, t1 - t0), sms),
             "tiles per CTA: min %d, max %d, total %d" % (min(t for _, _, t in ran), max(t for _, _, t in ran), sum(t for _, _, t in ran))]
    return "\n".join(lines)


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("workload")
    ap.add_argument("--cta", type=int, default=0, help="blockIdx.x of the traced CTA")
    ap.add_argument("--tile", type=int, default=0, help="first of the CTA's two traced tiles")
    ap.add_argument("--spans", action="store_true",
                    help="instead of the role timeline: when every CTA of a (warm) launch started and ended")
    args = ap.parse_args(argv)
    import torch
    from . import binding, inputs
    build_trace_library(args.cta, args.tile)
    binding.LIB_PATH = TRACE_LIB
    w = inputs.get(args.workload)
    dev = torch.device("cuda:0")
    q, k, v = [x.to(dev) for x in inputs.make_inputs(w)]
    binding.ave_attn_fwd(q, k, v, causal=w.causal, scale=w.scale)     # one launch: stamps of several would mix
    st, raw = binding.device_status()
    if st != binding.AVE_OK:
        raise RuntimeError("device status %d raw %#x" % (st, raw))
    L = binding.lib()
    if args.spans:
        n_ctas = 8192
        L.ave_attn_trace_read_spans.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.ave_attn_trace_read_spans.restype = ctypes.c_int
        L.ave_attn_trace_clear_spans.restype = ctypes.c_int
        for _ in range(3):   # the launch that is read is a warm one
            if L.ave_attn_trace_clear_spans() != 0:
                raise RuntimeError("ave_attn_trace_clear_spans failed")
            binding.ave_attn_fwd(q, k, v, causal=w.causal, scale=w.scale)
        sp = (ctypes.c_ulonglong * (3 * n_ctas))()
        if L.ave_attn_trace_read_spans(sp, n_ctas) != 0:
            raise RuntimeError("ave_attn_trace_read_spans failed")
        vals = list(sp)
        print(span_summary([tuple(vals[3 * i:3 * i + 3]) for i in range(n_ctas)],
                           torch.cuda.get_device_properties(0).multi_processor_count))
        return 0
    buf = (ctypes.c_longlong * (ROLES * ITERS * SLOTS))()
    L.ave_attn_trace_read.argtypes = [ctypes.c_void_p]
    L.ave_attn_trace_read.restype = ctypes.c_int
    if L.ave_attn_trace_read(buf) != 0:
        raise RuntimeError("ave_attn_trace_read failed")
    prev = {}
    for x, who, text in events(list(buf)):
        d = x - prev.get(who, x)
        prev[who] = x
        col = {"MMA": 0, "SM0": 1, "SM1": 2, "LD ": 3}[who]
        print("%9d  %s%-4s +%-6d %s" % (x, " " * (26 * col), who, d, text))
    return 0


if __name__ == "__main__":
    sys.exit(main())
