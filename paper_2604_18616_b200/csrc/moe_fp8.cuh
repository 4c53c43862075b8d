// Block-quantised FP8 fused mixture-of-experts layer for sm_100a (the paper's third kernel family, Section 9:
// DeepSeek-V3.2's block-quantised FP8 configuration; "quantize up-projection intermediates to FP8", "preserve
// blockwise quantization, route tokens through sorted expert maps, and group accesses for coalescing").
//
// Format: E4M3 codes; activations carry one fp32 scale per (token, 128 channels), weights one per 128 x 128
// block.  Steps of one call (all on the caller's stream, scratch in the caller's workspace):
//   1. moe_count_kernel / moe_scatter_kernel: (token, k) pairs sorted by expert; every expert's rows start on
//      a multiple of 128, so a 128-row tile of the sorted order belongs to one expert
//   2. moe_gather_kernel: the tokens' codes and scales copied into the sorted order (padding rows are zero)
//   3. moe_gemm_fp8_kernel: h = x W13^T, rows x 2F, fp32       (grouped by expert, block-scaled, tensor cores)
//   4. moe_act_quant_kernel: a = silu(gate) * up, requantised to E4M3 per 128 columns, fp32 scale
//   5. moe_gemm_fp8_kernel: o = w * (a W2^T), rows x C, fp32   (w: the pair's routing weight)
//   6. moe_combine_kernel: y[t] = sum over the token's K rows of o, rounded to bf16
//
// The GEMM: persistent CTAs over 128 x 256 output tiles; K is streamed in blocks of 128 (one scale block)
// through a TMA ring; each block is four M128 x N256 x K32 tcgen05 MMAs (kind::f8f6f4) into one of two TMEM
// accumulators, which the epilogue warps read out and add, multiplied by the block's scales, to fp32
// registers (the accumulation across scale blocks cannot stay in the tensor core: every block has its own
// factor).  Rows are TMEM lanes; two epilogue threads per row, 128 columns (one weight scale block) each.
//
//   warp 0       producer: TMA loads of the A and B blocks
//   warp 1       MMA issuer
//   warp 2       TMEM allocation / release
//   warp 3       -
//   warps 4..11  epilogue (thread = output row x half of the tile's columns)
#pragma once

#include <cuda_bf16.h>

#include "attn_common.cuh"

namespace ave {

constexpr int kMoeGroup = 128;  // channels per activation scale, rows and columns per weight scale block

struct MoeGemmCfg {
    static constexpr int kThreads = 384;
    static constexpr int kTile = 128;                          // rows of an output tile; K block; columns per epilogue thread
    static constexpr int kTileN = 256;                         // columns of an output tile
    static constexpr int kStages = 4;
    static constexpr int kABytes = kTile * kMoeGroup;          // 16 KB of E4M3
    static constexpr int kBBytes = kTileN * kMoeGroup;         // 32 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStageCBytes = 8 * 32 * 128;          // result staging: 32 rows x 32 fp32 per epilogue warp
    static constexpr int kSmemBytes = kStages * kStageBytes + kStageCBytes + 1024;
    static constexpr int kAccs = 2;                            // TMEM accumulators of 256 columns
    static constexpr uint32_t kTmemCols = kAccs * kTileN;
    // The epilogue threads hold 128 fp32 sums plus two 32-column chunks in flight: they take registers from the
    // producer / MMA warpgroup (setmaxnreg moves them inside the CTA's allocation of kThreads x kRegsAtLaunch;
    // the build and the launch code check the compiled image against this split).
    static constexpr int kRegsLight = 40, kRegsEpilogue = 232, kRegsAtLaunch = 168;
    static_assert(128 * kRegsLight + 256 * kRegsEpilogue <= kThreads * kRegsAtLaunch, "register split exceeds the CTA's allocation");
};

struct MoeGemmParams {
    const float *a_scale;     // [rows, K/128]
    const float *b_scale;     // [E, N/128, K/128]
    const int *tile_expert;   // [rows/128]: expert of each 128-row tile of the sorted order, -1 = unused tile
    const float *row_weight;  // [rows] or NULL: factor applied to every output row
    float *out;               // [rows, N] fp32
    int tiles_m, tiles_n;     // rows / 128, ceil(N / 256)
    int nblk;                 // N / 128: weight scale blocks along N
    int kb;                   // K / 128
    int N;
};

// tcgen05 instruction descriptor, kind::f8f6f4: fp32 accumulator, E4M3 A and B, both K-major.
__host__ __device__ constexpr uint32_t make_idesc_e4m3(int m, int n) {
    return (1u << 4)                       // D format: f32
           | (0u << 7)                     // A format: E4M3
           | (0u << 10)                    // B format: E4M3
           | (uint32_t(n >> 3) << 17)      // N / 8
           | (uint32_t(m >> 4) << 24);     // M / 16
}

__device__ __forceinline__ void umma_f8_ss_words(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                 uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .b64 da, db;\n"
        "setp.ne.b32 p, %6, 0;\n"
        "mov.b64 da, {%1, %2};\n"
        "mov.b64 db, {%3, %4};\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %5, p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Output tile number -> (row tile, column tile): groups of 4 row tiles (about one expert's rows at the paper's
// sizes), column-major inside a group, so that CTAs at work together share a few experts' weights in L2.
__device__ __forceinline__ void moe_tile_coords(int id, const MoeGemmParams &p, int &bm, int &bn) {
    constexpr int kGroupM = 4;
    const int per_group = kGroupM * p.tiles_n;
    const int grp = id / per_group;
    const int rem = id - grp * per_group;
    const int m0 = grp * kGroupM;
    const int gm = min(kGroupM, p.tiles_m - m0);
    bn = rem / gm;
    bm = m0 + (rem - bn * gm);
}

// tm_a: A codes [rows, K] as {K, rows, 1, 1}, boxes of 128 bytes x 128 rows; tm_b: B codes [E, N, K] as
// {K, N, E, 1}, boxes of 128 bytes x 256 rows (rows beyond N read as zero); tm_c: the fp32 result [rows, N] as
// {N, rows, 1, 1}, boxes of 32 columns x 32 rows (a thread-per-row store of fp32 rows would touch 32 rows per
// instruction, one sector each: measured, that cost more than the tile's products).
__global__ void __launch_bounds__(384, 1)
moe_gemm_fp8_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_c, const MoeGemmParams p) {
    using Cfg = MoeGemmCfg;
    constexpr int NS = Cfg::kStages, NA = Cfg::kAccs;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[NS], bar_empty[NS], bar_acc_full[NA], bar_acc_empty[NA], bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t sRing = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (tid == 0) {
        abort_flag = (*reinterpret_cast<volatile unsigned int *>(&g_device_status) != 0) ? 1 : 0;
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int a = 0; a < NA; ++a) {
            mbar_init(smem_u32(&bar_acc_full[a]), 1);
            mbar_init(smem_u32(&bar_acc_empty[a]), 8);  // one arrival per epilogue warp
        }
        mbar_init(smem_u32(&bar_drain), 1);
        fence_mbar_init();
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const bool poisoned = abort_flag != 0;

    auto wait_bar = [&](uint64_t *bar, uint32_t parity, unsigned code) -> bool {
        const bool r = mbar_wait_bounded(smem_u32(bar), parity, &abort_flag, code);
        return __all_sync(0xffffffffu, r);
    };

    const int n_tiles = p.tiles_m * p.tiles_n;

    if (poisoned) {
        // nothing: fall through to the common exit
    } else if (warp < 4) {
      setmaxnreg_dec<Cfg::kRegsLight>();
      if (warp == 0) {
        // =============================== producer ===============================
        const bool leader = elect_one();
        if (leader) {
            tma_prefetch_desc(&tm_a);
            tma_prefetch_desc(&tm_b);
        }
        bool ok = true;
        int ring = 0;  // K blocks loaded so far
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            int bm, bn;
            moe_tile_coords(tile, p, bm, bn);
            const int e = p.tile_expert[bm];
            if (e < 0) continue;  // a row tile beyond the sorted rows
            for (int kb = 0; kb < p.kb && ok; ++kb, ++ring) {
                const int slot = ring % NS, round = ring / NS;
                if (round > 0) {
                    ok = wait_bar(&bar_empty[slot], (round - 1) & 1, STATUS_TIMEOUT_SLOT);
                    if (!ok) break;
                }
                if (leader) {
                    const uint32_t bar = smem_u32(&bar_full[slot]);
                    const uint32_t dst = sRing + slot * Cfg::kStageBytes;
                    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    tma_load_4d(dst, &tm_a, bar, kb * kMoeGroup, bm * Cfg::kTile, 0, 0);
                    tma_load_4d(dst + Cfg::kABytes, &tm_b, bar, kb * kMoeGroup, bn * Cfg::kTileN, e, 0);
                }
            }
        }
        if (!ok) {
            for (int it = max(0, ring - NS); it < ring; ++it)
                for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_full[it % NS]), (it / NS) & 1); ++w) {}
        }
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        const bool leader = elect_one();
        constexpr uint32_t idesc = make_idesc_e4m3(Cfg::kTile, Cfg::kTileN);
        constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);  // rows of 128 bytes, 8-row atoms of 1024 bytes
        constexpr uint32_t hi = uint32_t(desc_kmajor >> 32), lo = uint32_t(desc_kmajor);
        bool ok = true;
        int ring = 0;  // K blocks issued so far = accumulators filled so far
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            int bm, bn;
            moe_tile_coords(tile, p, bm, bn);
            if (p.tile_expert[bm] < 0) continue;
            for (int kb = 0; kb < p.kb && ok; ++kb, ++ring) {
                const int slot = ring % NS, acc = ring % NA;
                if (ring >= NA) {  // the epilogue must have read this accumulator's previous block out of TMEM
                    ok = wait_bar(&bar_acc_empty[acc], ((ring / NA) - 1) & 1, STATUS_TIMEOUT_SOFTMAX);
                    if (!ok) break;
                }
                ok = wait_bar(&bar_full[slot], (ring / NS) & 1, STATUS_TIMEOUT_LOAD);
                if (!ok) break;
                tc_fence_after();
                if (leader) {
                    const uint32_t a_lo = lo | ((sRing + slot * Cfg::kStageBytes) >> 4);
                    const uint32_t b_lo = lo | ((sRing + slot * Cfg::kStageBytes + Cfg::kABytes) >> 4);
                    const uint32_t d_tmem = tmem + acc * Cfg::kTileN;
#pragma unroll
                    for (int kk = 0; kk < kMoeGroup / 32; ++kk)  // K = 32 bytes per instruction
                        umma_f8_ss_words(d_tmem, a_lo + ((kk * 32) >> 4), hi, b_lo + ((kk * 32) >> 4), hi, idesc, kk > 0);
                    umma_commit(smem_u32(&bar_empty[slot]));
                    umma_commit(smem_u32(&bar_acc_full[acc]));
                }
            }
        }
        if (!ok) {  // abandoned: let the MMAs already issued finish before TMEM is released
            if (leader) umma_commit(smem_u32(&bar_drain));
            for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_drain), 0); ++w) {}
        }
      }
    } else {
        // =============================== epilogue ===============================
        setmaxnreg_inc<Cfg::kRegsEpilogue>();
        const int wq = warp & 3;           // TMEM lane quadrant of this warp
        const int half = (warp - 4) >> 2;  // which 128 of the tile's 256 columns
        const uint32_t lane_sel = uint32_t(wq * 32) << 16;
        const uint32_t sC = sRing + NS * Cfg::kStageBytes + (warp - 4) * (32 * 128);  // this warp's 32 staging rows
        bool store_pending = false;  // (lane 0) a TMA store may still be reading the staging rows
        bool ok = true;
        int ring = 0;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            int bm, bn;
            moe_tile_coords(tile, p, bm, bn);
            const int e = p.tile_expert[bm];
            if (e < 0) continue;
            const int row = bm * Cfg::kTile + wq * 32 + lane;
            const int nb = bn * 2 + half;              // this thread's weight scale block along N
            const bool live = nb < p.nblk;             // (the last tile's second half lies beyond N when N % 256 == 128)
            const float *sa = p.a_scale + size_t(row) * p.kb;
            const float *sb = p.b_scale + (size_t(e) * p.nblk + (live ? nb : 0)) * p.kb;
            float acc[Cfg::kTile];
#pragma unroll
            for (int c = 0; c < Cfg::kTile; ++c) acc[c] = 0.f;
            float s_next = sa[0] * sb[0];
            for (int kb = 0; kb < p.kb && ok; ++kb, ++ring) {
                const float s = s_next;
                if (kb + 1 < p.kb) s_next = sa[kb + 1] * sb[kb + 1];  // fetched while this block is awaited
                const int a = ring % NA;
                ok = wait_bar(&bar_acc_full[a], (ring / NA) & 1, STATUS_TIMEOUT_MMA);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_acc = tmem + a * Cfg::kTileN + half * Cfg::kTile + lane_sel;
                // 32 columns at a time, the next chunk's load in flight while this chunk is added up
                uint32_t v[2][32];
                tmem_ld_x32(t_acc, v[0]);
#pragma unroll
                for (int c = 0; c < Cfg::kTile / 32; ++c) {
                    tmem_wait_ld();
                    if (c + 1 < Cfg::kTile / 32) {
                        tmem_ld_x32(t_acc + (c + 1) * 32, v[(c + 1) & 1]);
                    } else {  // the block's products are in registers: the accumulator is free
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[a]));
                    }
#pragma unroll
                    for (int x = 0; x < 32; ++x) acc[c * 32 + x] = fmaf(__uint_as_float(v[c & 1][x]), s, acc[c * 32 + x]);
                }
            }
            if (!ok) break;
            if (!live) continue;
            const float w = p.row_weight ? p.row_weight[row] : 1.f;
            // 32 columns at a time through this warp's staging rows (128 bytes each, 128-byte swizzle) and out by TMA
#pragma unroll
            for (int c = 0; c < Cfg::kTile / 32; ++c) {
                if (store_pending) {
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                }
#pragma unroll
                for (int x = 0; x < 32; x += 4) {
                    const uint32_t addr = sC + lane * 128 + ((uint32_t(x >> 2) ^ uint32_t(lane & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr),
                                 "r"(__float_as_uint(acc[c * 32 + x] * w)), "r"(__float_as_uint(acc[c * 32 + x + 1] * w)),
                                 "r"(__float_as_uint(acc[c * 32 + x + 2] * w)), "r"(__float_as_uint(acc[c * 32 + x + 3] * w))
                                 : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_4d(&tm_c, sC, nb * Cfg::kTile + c * 32, bm * Cfg::kTile + wq * 32, 0, 0);
                    tma_store_commit();
                }
                store_pending = true;
            }
        }
        if (lane == 0 && store_pending) tma_store_wait_all();
    }

    // ---- common exit: every thread arrives, then TMEM is released
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, Cfg::kTmemCols);
}

// ------------------------------------------------------------------ routing: sort (token, k) pairs by expert
// One CTA: counts per expert, padded offsets (every expert starts on a multiple of 128 rows), the expert of every
// 128-row tile (-1 beyond the last used tile), pair_of = -1 for every row (padding until the scatter fills it in).
__global__ void moe_count_kernel(const int *__restrict__ ids, int n_pairs, int E, int rows_cap, int *expert_off,
                                 int *cursor, int *tile_expert, int *pair_of, int *bad_id) {
    extern __shared__ int counts[];  // E
    for (int e = threadIdx.x; e < E; e += blockDim.x) counts[e] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n_pairs; i += blockDim.x) {
        const int e = ids[i];
        if (e >= 0 && e < E) atomicAdd(&counts[e], 1);
        else *bad_id = 1;
    }
    for (int r = threadIdx.x; r < rows_cap; r += blockDim.x) pair_of[r] = -1;
    __syncthreads();
    if (threadIdx.x == 0) {
        int off = 0;
        for (int e = 0; e < E; ++e) {
            expert_off[e] = off;
            cursor[e] = 0;
            const int tiles = (counts[e] + 127) / 128;
            for (int t = 0; t < tiles; ++t) tile_expert[off / 128 + t] = e;
            off += tiles * 128;
        }
        expert_off[E] = off;
        for (int t = off / 128; t < rows_cap / 128; ++t) tile_expert[t] = -1;
    }
}

__global__ void moe_scatter_kernel(const int *__restrict__ ids, int n_pairs, int E, const int *__restrict__ expert_off,
                                   int *cursor, int *row_of, int *pair_of) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pairs) return;
    const int e = ids[i];
    if (e < 0 || e >= E) {
        row_of[i] = -1;
        return;
    }
    const int row = expert_off[e] + atomicAdd(&cursor[e], 1);
    row_of[i] = row;
    pair_of[row] = i;
}

// Codes and scales of every sorted row's token (zeros for padding rows), and the row's routing weight.
// One CTA per row; C / 16 threads' worth of 16-byte copies.
__global__ void moe_gather_kernel(const uint8_t *__restrict__ xq, const float *__restrict__ sx, const float *__restrict__ wts,
                                  const int *__restrict__ pair_of, const int *__restrict__ tile_expert, int C, int K,
                                  uint8_t *xq_s, float *sx_s, float *w_s) {
    const int row = blockIdx.x;
    if (tile_expert[row / 128] < 0) return;  // beyond the sorted rows: never read
    const int pair = pair_of[row];
    const int CG = C / kMoeGroup;
    uint4 *dst = reinterpret_cast<uint4 *>(xq_s + size_t(row) * C);
    if (pair < 0) {
        for (int i = threadIdx.x; i < C / 16; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
        for (int i = threadIdx.x; i < CG; i += blockDim.x) sx_s[size_t(row) * CG + i] = 0.f;
        if (threadIdx.x == 0) w_s[row] = 0.f;
        return;
    }
    const int t = pair / K;
    const uint4 *src = reinterpret_cast<const uint4 *>(xq + size_t(t) * C);
    for (int i = threadIdx.x; i < C / 16; i += blockDim.x) dst[i] = src[i];
    for (int i = threadIdx.x; i < CG; i += blockDim.x) sx_s[size_t(row) * CG + i] = sx[size_t(t) * CG + i];
    if (threadIdx.x == 0) w_s[row] = wts[pair];
}

// Two fp32 values -> two E4M3 codes (round to nearest even, saturating at +-448); `lo` lands in bits 0..7.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// a = silu(gate) * up in fp32, requantised per group of 128 columns: one warp per (row, group), four columns per
// lane.  s = max|a| / 448 and a / s are fp32 divisions rounded to nearest, as the format's definition has them.
__global__ void moe_act_quant_kernel(const float *__restrict__ h, const int *__restrict__ tile_expert, int F, int rows,
                                     uint8_t *aq, float *sa) {
    const int FG = F / kMoeGroup;
    const long long wid = (long long)blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
    if (wid >= (long long)rows * FG) return;
    const int row = int(wid / FG), g = int(wid - (long long)row * FG);
    if (tile_expert[row / 128] < 0) return;
    const int lane = threadIdx.x & 31;
    const float4 gate = reinterpret_cast<const float4 *>(h + size_t(row) * 2 * F + g * kMoeGroup)[lane];
    const float4 up = reinterpret_cast<const float4 *>(h + size_t(row) * 2 * F + F + g * kMoeGroup)[lane];
    float a[4];
    a[0] = __fdiv_rn(gate.x, 1.f + expf(-gate.x)) * up.x;
    a[1] = __fdiv_rn(gate.y, 1.f + expf(-gate.y)) * up.y;
    a[2] = __fdiv_rn(gate.z, 1.f + expf(-gate.z)) * up.z;
    a[3] = __fdiv_rn(gate.w, 1.f + expf(-gate.w)) * up.w;
    float amax = fmaxf(fmaxf(fabsf(a[0]), fabsf(a[1])), fmaxf(fabsf(a[2]), fabsf(a[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float s = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
    const uint32_t c01 = cvt_e4m3x2(__fdiv_rn(a[0], s), __fdiv_rn(a[1], s));
    const uint32_t c23 = cvt_e4m3x2(__fdiv_rn(a[2], s), __fdiv_rn(a[3], s));
    reinterpret_cast<uint32_t *>(aq + size_t(row) * F + g * kMoeGroup)[lane] = c01 | (c23 << 16);
    if (lane == 0) sa[size_t(row) * FG + g] = s;
}

// y[t, :] = sum over the token's K sorted rows of o (already weighted), in the order k = 0..K-1, rounded to bf16.
__global__ void moe_combine_kernel(const float *__restrict__ o, const int *__restrict__ row_of, int T, int C, int K,
                                   __nv_bfloat16 *y) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int per_row = C / 4;
    if (idx >= (long long)T * per_row) return;
    const int t = int(idx / per_row), c4 = int(idx - (long long)t * per_row);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < K; ++k) {
        const int row = row_of[t * K + k];
        if (row < 0) continue;
        const float4 v = reinterpret_cast<const float4 *>(o + size_t(row) * C)[c4];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    uint2 out;
    out.x = pack_bf16x2(acc.x, acc.y);
    out.y = pack_bf16x2(acc.z, acc.w);
    reinterpret_cast<uint2 *>(y + size_t(t) * C)[c4] = out;
}

}  // namespace ave
