"""Seeded synthetic attention workloads and their bookkeeping.

This module only draws random tensors and counts work; it contains none of the
attention arithmetic.  It is the one module that both the CUDA path's tests and
the CPU oracle's tests may import.

Generation rule (every workload): one CPU ``torch.Generator`` seeded with the
workload's seed draws fp32 Q, then K, then V, in that order; the stated
transform is applied in fp32; the result is rounded to bf16 (round to nearest
even).  The shapes mirror the paper's evaluation of attention (Section 9:
causal bf16 grouped-query prefill, head dimension 128, sequence lengths from
1024 to 16384) plus a tiny case and a wide non-causal case.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Hkv: int
    Sq: int
    Sk: int
    D: int
    causal: bool
    seed: int
    dist: str = "normal"          # "normal": N(0,1); "uniform": U[-2, 2]
    peaked_every: int = 0          # >0: key rows j % peaked_every == 0 are multiplied by 4
    note: str = ""

    @property
    def scale(self) -> float:
        """1/sqrt(D), rounded to fp32 (the value handed to the library)."""
        return float(torch.tensor(1.0 / math.sqrt(self.D), dtype=torch.float32).item())

    @property
    def G(self) -> int:
        return self.H // self.Hkv


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", 1, 2, 2, 128, 128, 64, False, 0,
                        note="tiny non-causal case the oracle finishes instantly"),
    "c2_mha_prefill": Workload("c2_mha_prefill", 4, 32, 32, 2048, 2048, 128, True, 1,
                               note="causal multi-head prefill"),
    "c3_gqa_prefill": Workload("c3_gqa_prefill", 2, 64, 8, 4096, 4096, 128, True, 2,
                               note="causal grouped-query prefill, 8 query heads per KV head"),
    "c4_long_context": Workload("c4_long_context", 1, 32, 8, 16384, 16384, 128, True, 3,
                                peaked_every=64,
                                note="long causal prefill, every 64th key row x4 (peaked softmax rows)"),
    "c5_wide_noncausal": Workload("c5_wide_noncausal", 8, 16, 16, 8192, 8192, 64, False, 4,
                                  dist="uniform", note="encoder-style, head dim 64, U[-2,2]"),
}

# The paper's own attention workload (Section 9): causal bf16 GQA, batch 16,
# 8 query heads, 1 KV head, head dimension 128, N in {1024..16384}.
for _n in (1024, 2048, 4096, 8192, 16384):
    WORKLOADS["paper_gqa_n%d" % _n] = Workload(
        "paper_gqa_n%d" % _n, 16, 8, 1, _n, _n, 128, True, 100 + _n // 1024,
        note="the paper's evaluation shape (LLaMA-3 70B prefill under 8-way TP)")


# Head dimensions above 128 (the single-sub-tile kernel with 256 output columns in TMEM).
WORKLOADS["d256_gqa_prefill"] = Workload("d256_gqa_prefill", 2, 32, 8, 4096, 4096, 256, True, 301,
                                         note="causal grouped-query prefill, head dimension 256")
WORKLOADS["d192_gqa_prefill"] = Workload("d192_gqa_prefill", 2, 32, 8, 4096, 4096, 192, True, 302,
                                         note="causal grouped-query prefill, head dimension 192 (computed as 256)")

# Decode: one new query token per sequence against a long key/value cache (the split-KV entry point);
# bound by reading K and V once from HBM.
for _name, _b, _h, _hkv, _sk, _seed in (("decode_mha_b8_k8192", 8, 32, 32, 8192, 201),
                                        ("decode_gqa_b8_k16384", 8, 32, 8, 16384, 202),
                                        ("decode_gqa_b1_k65536", 1, 32, 8, 65536, 203),
                                        ("decode_gqa_b64_k4096", 64, 32, 8, 4096, 204)):
    WORKLOADS[_name] = Workload(_name, _b, _h, _hkv, 1, _sk, 128, True, _seed,
                                note="decode step: one query row per sequence, split-KV")


def get(name: str) -> Workload:
    return WORKLOADS[name]


def small_variant(w: Workload, **kw) -> Workload:
    """A same-recipe workload with some fields overridden (tests use this)."""
    return replace(w, **kw)


def make_inputs(w: Workload):
    """(q, k, v) as CPU bf16 tensors [B,H,Sq,D], [B,Hkv,Sk,D], [B,Hkv,Sk,D]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    shapes = [(w.B, w.H, w.Sq, w.D), (w.B, w.Hkv, w.Sk, w.D), (w.B, w.Hkv, w.Sk, w.D)]
    out = []
    for idx, shp in enumerate(shapes):
        if w.dist == "normal":
            x = torch.randn(shp, generator=g, dtype=torch.float32)
        elif w.dist == "uniform":
            x = torch.rand(shp, generator=g, dtype=torch.float32) * 4.0 - 2.0
        else:
            raise ValueError("unknown dist %r" % w.dist)
        if idx == 1 and w.peaked_every > 0:
            x[:, :, :: w.peaked_every, :] *= 4.0
        out.append(x.to(torch.bfloat16))
    return tuple(out)


def tensor_sha256(t: torch.Tensor) -> str:
    return hashlib.sha256(t.contiguous().view(torch.uint8).numpy().tobytes()).hexdigest()


def visible_pairs(w: Workload) -> int:
    """Number of (query, key) pairs the mask leaves visible, over all b, h."""
    if not w.causal:
        per_head = w.Sq * w.Sk
    else:
        off = w.Sk - w.Sq
        per_head = sum(min(w.Sk, max(0, i + 1 + off)) for i in range(w.Sq))
    return w.B * w.H * per_head


def attn_flops(w: Workload) -> float:
    """Counted FLOPs: 4*B*H*Sq*Sk*D, halved when causal."""
    f = 4.0 * w.B * w.H * w.Sq * w.Sk * w.D
    return f * 0.5 if w.causal else f


def min_hbm_bytes(w: Workload) -> int:
    """|Q| + |K| + |V| + |O| + |LSE| in bytes: every tensor touched once."""
    q = w.B * w.H * w.Sq * w.D * 2
    kv = 2 * w.B * w.Hkv * w.Sk * w.D * 2
    o = q
    lse = w.B * w.H * w.Sq * 4
    return q + kv + o + lse


def sample_rows(w: Workload, n_random: int, seed: int = 12345, tile: int = 128):
    """Rows (b, h, i) for sampled parity on large workloads.

    Every (b, h) contributes the rows next to each multiple of ``tile`` near
    the start, middle and end; ``n_random`` further rows are uniform over
    (b, h, i).
    """
    edge = set()
    for base in (0, tile, 2 * tile, (w.Sq // 2 // tile) * tile, ((w.Sq - 1) // tile) * tile):
        for d in (-1, 0, 1):
            i = base + d
            if 0 <= i < w.Sq:
                edge.add(i)
    edge.add(w.Sq - 1)
    rows = [(b, h, i) for b in range(w.B) for h in range(w.H) for i in sorted(edge)]
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    if n_random > 0:
        rb = torch.randint(0, w.B, (n_random,), generator=g)
        rh = torch.randint(0, w.H, (n_random,), generator=g)
        ri = torch.randint(0, w.Sq, (n_random,), generator=g)
        rows += list(zip(rb.tolist(), rh.tolist(), ri.tolist()))
    return rows


def make_gemm_inputs(M: int, N: int, K: int, seed: int):
    """A [M, K] and B [N, K] for the matrix-product workload (the paper's Section 9: bf16 matrices
    with normally distributed entries): one CPU generator draws fp32 A, then B, N(0,1), rounded to bf16."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    a = torch.randn((M, K), generator=g, dtype=torch.float32).to(torch.bfloat16)
    b = torch.randn((N, K), generator=g, dtype=torch.float32).to(torch.bfloat16)
    return a, b


# ------------------------------------------------------------------ fused MoE (block-quantised FP8)
@dataclass(frozen=True)
class MoeWorkload:
    """The paper's fused-MoE configuration (Section 9): model dimension C, intermediate dimension F, top-k K,
    E experts on this GPU; T tokens whose K routed experts all live on this GPU."""
    name: str
    T: int
    C: int = 7168
    F: int = 2048
    E: int = 32
    K: int = 4
    seed: int = 400


MOE_WORKLOADS = {n: MoeWorkload(n, t, seed=400 + i) for i, (n, t) in enumerate(
    (("moe_t256", 256), ("moe_t1024", 1024), ("moe_t4096", 4096), ("moe_t8192", 8192), ("moe_t16384", 16384)))}


# Exponent field of a random E4M3 code, looked up with a uniform byte: most values within a factor of 8 below the
# block maximum, as in block-quantised Gaussian data.  (A table of bit patterns; nothing here evaluates the format.)
_EXPO_OF_BYTE = torch.tensor([15] * 26 + [14] * 82 + [13] * 72 + [12] * 38 + [11] * 20 + [10] * 10 + [9] * 5 + [8] * 3,
                             dtype=torch.uint8)
assert _EXPO_OF_BYTE.numel() == 256


def _fp8_codes(g: torch.Generator, shape, group_axis_len: int):
    """Random E4M3 bit patterns shaped like block-quantised Gaussian data: exponent field from the table above,
    mantissa and sign uniform; the first element of every group of 128 along the last axis is the block maximum
    (+-448, code 0x7e), as it is after scaling a block by its largest magnitude.  No NaN pattern is produced."""
    out = torch.empty(shape, dtype=torch.uint8)
    flat = out.view(-1)
    n = flat.numel()
    step = 1 << 26
    for lo in range(0, n, step):
        m = min(step, n - lo)
        expo = _EXPO_OF_BYTE[torch.randint(0, 256, (m,), generator=g, dtype=torch.int64)]
        low = torch.randint(0, 16, (m,), generator=g, dtype=torch.uint8)       # sign bit and mantissa
        mant = low & 7
        mant = torch.where((expo == 15) & (mant == 7), torch.zeros_like(mant), mant)   # 0x7f would be NaN
        flat[lo:lo + m] = ((low >> 3) << 7) | (expo << 3) | mant
    lead = out[..., ::group_axis_len]
    out[..., ::group_axis_len] = (lead & 0x80) | 0x7E
    return out


def _expert_codes(g: torch.Generator, E: int, rows: int, cols: int):
    """[E, rows, cols] codes: four experts are drawn; expert e repeats expert e % 4 rotated by 128 * (e // 4) columns
    (drawing 1.4 G independent codes takes most of a minute; the experts' scales are all different)."""
    base = _fp8_codes(g, (min(E, 4), rows, cols), 128)
    out = torch.empty((E, rows, cols), dtype=torch.uint8)
    for e in range(E):
        out[e] = torch.roll(base[e % 4], shifts=128 * (e // 4), dims=1) if e >= 4 else base[e]
    return out


_MOE_WEIGHTS = {}


def _moe_weights(C: int, F: int, E: int):
    """The layer's quantised weights: one set per (C, F, E), shared by the workloads of every token count (seed 4000)."""
    key = (C, F, E)
    if key not in _MOE_WEIGHTS:
        g = torch.Generator(device="cpu")
        g.manual_seed(4000)
        w13q = _expert_codes(g, E, 2 * F, C)
        s13 = ((0.8 + 0.4 * torch.rand((E, 2 * F // 128, C // 128), generator=g)) * (2.8 / 448.0 / math.sqrt(C))).float()
        w2q = _expert_codes(g, E, C, F)
        s2 = ((0.8 + 0.4 * torch.rand((E, C // 128, F // 128), generator=g)) * (2.8 / 448.0 / math.sqrt(F))).float()
        _MOE_WEIGHTS.clear()      # one set at a time: the paper's configuration is 1.4 GB
        _MOE_WEIGHTS[key] = (w13q, s13, w2q, s2)
    return _MOE_WEIGHTS[key]


def make_moe_inputs(w: MoeWorkload):
    """(xq u8 [T,C], sx f32 [T,C/128], w13q u8 [E,2F,C], s13 f32 [E,2F/128,C/128], w2q u8 [E,C,F],
    s2 f32 [E,C/128,F/128], ids i32 [T,K], wts f32 [T,K]) as CPU tensors.  Scales are drawn so that the
    dequantised activations look like N(0,1) data and the dequantised weights like N(0, 1/fan_in) data; every
    token gets K distinct experts and positive routing weights that sum to one."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    T, C, F, E, K = w.T, w.C, w.F, w.E, w.K
    xq = _fp8_codes(g, (T, C), 128)
    sx = ((0.8 + 0.4 * torch.rand((T, C // 128), generator=g)) * (2.8 / 448.0)).float()
    w13q, s13, w2q, s2 = _moe_weights(C, F, E)
    ids = torch.argsort(torch.rand((T, E), generator=g), dim=1)[:, :K].to(torch.int32).contiguous()
    raw = 0.1 + torch.rand((T, K), generator=g)
    wts = (raw / raw.sum(dim=1, keepdim=True)).to(torch.float32)
    return xq, sx, w13q, s13, w2q, s2, ids, wts


def moe_flops(w: MoeWorkload) -> float:
    """Counted FLOPs: 2 * T * K * (2F*C + C*F)."""
    return 2.0 * w.T * w.K * (2.0 * w.F * w.C + 1.0 * w.C * w.F)
