// Dense bf16 GEMM for sm_100a: C[M, N] = A[M, K] * B[N, K]^T (or A[M, K] * B[K, N]),
// fp32 accumulation in TMEM, bf16 result.  (The paper's first evaluated kernel family, Section 9:
// square bf16 matrices with normally distributed entries.)
//
// Persistent CTAs, one per SM, each walking output tiles of 128 x 256 (128 x 128
// for small products) in a
// static order.  Inside a tile the K dimension is streamed in slices of 64
// through a ring of shared-memory stages filled by TMA; one thread issues
// M128 x N256 x K16 tcgen05 MMAs into one of two TMEM accumulators, so the
// epilogue of a tile (TMEM -> registers -> bf16 -> shared -> TMA store)
// overlaps the main loop of the next one.
//
//   warp 0      producer: TMA loads of the A and B slices
//   warp 1      MMA issuer
//   warp 2      TMEM allocation / release
//   warp 3      -
//   warps 4..7  epilogue (thread = accumulator row = TMEM lane)
//
// Rows and columns outside the matrices are zero-filled by the loads and
// clipped by the stores, so M, N and K need not be multiples of the tile.
#pragma once

#include "attn_common.cuh"

namespace ave {

// TN = 256 is the tile for large products; TN = 128 halves the tile for products with fewer 128 x 256
// tiles than SMs, where more, shorter tiles finish earlier.
template <int TN>
struct GemmCfg {
    static_assert(TN == 128 || TN == 256, "tile widths the kernel is instantiated for");
    static constexpr int kThreads = 256;
    static constexpr int kTileM = 128, kTileN = TN, kSliceK = 64;
    static constexpr int kStages = (TN == 256) ? 4 : 6;
    static constexpr int kABytes = kTileM * kSliceK * 2;          // 16 KB
    static constexpr int kBBytes = kTileN * kSliceK * 2;          // 32 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOutBoxRows = 32;                        // each epilogue warp stores its own 32 rows
    static constexpr int kStageCBytes = 4 * kOutBoxRows * 128;    // C staging: 32 rows x 64 columns per epilogue warp
    static constexpr int kSmemBytes = kStages * kStageBytes + kStageCBytes + 1024;
    static constexpr uint32_t kTmemCols = 2 * TN;                 // two accumulators of TN columns
};

struct GemmParams {
    int M, N, K;
    int tiles_m, tiles_n;  // output tiles along M and N
    int group_m;           // tiles along M walked together before moving along N (L2 reuse of the B tiles)
};

// Output tile number `id` -> (block row, block column): groups of `group_m` block rows, column-major inside a
// group, so that CTAs working at the same time share a few A row blocks and neighbouring B column blocks.
__device__ __forceinline__ void gemm_tile_coords(int id, const GemmParams &p, int &bm, int &bn) {
    const int per_group = p.group_m * p.tiles_n;
    const int grp = id / per_group;
    const int rem = id - grp * per_group;
    const int m0 = grp * p.group_m;
    const int gm = min(p.group_m, p.tiles_m - m0);
    bn = rem / gm;
    bm = m0 + (rem - bn * gm);
}

// B_NMAJOR = false: B is [N, K] with K contiguous (C = A * B^T).  B_NMAJOR = true: B is [K, N] with N
// contiguous (C = A * B); its slice then lands in shared memory as 64-column boxes of 64 K-rows each and is
// read through an MN-major descriptor, so neither form needs a transposition.
template <int TN, bool B_NMAJOR>
__global__ void __launch_bounds__(256, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
    using Cfg = GemmCfg<TN>;
    constexpr int NS = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[NS], bar_empty[NS], bar_acc_full[2], bar_acc_empty[2], bar_drain;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sRing = smem_base;
    const uint32_t sStage = sRing + NS * Cfg::kStageBytes;

    if (tid == 0) {
        abort_flag = (*reinterpret_cast<volatile unsigned int *>(&g_device_status) != 0) ? 1 : 0;
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bar_acc_full[a]), 1);
            mbar_init(smem_u32(&bar_acc_empty[a]), 4);  // one arrival per epilogue warp
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
    const int n_slices = (p.K + Cfg::kSliceK - 1) / Cfg::kSliceK;

    if (poisoned) {
        // nothing: fall through to the common exit
    } else if (warp == 0) {
        // =============================== producer ===============================
        const bool leader = elect_one();
        if (leader) {
            tma_prefetch_desc(&tm_a);
            tma_prefetch_desc(&tm_b);
        }
        bool ok = true;
        int ring = 0;  // slices loaded so far
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            int bm, bn;
            gemm_tile_coords(tile, p, bm, bn);
            for (int ks = 0; ks < n_slices && ok; ++ks, ++ring) {
                const int slot = ring % NS, round = ring / NS;
                if (round > 0) {
                    ok = wait_bar(&bar_empty[slot], (round - 1) & 1, STATUS_TIMEOUT_SLOT);
                    if (!ok) break;
                }
                if (leader) {
                    const uint32_t bar = smem_u32(&bar_full[slot]);
                    const uint32_t dst = sRing + slot * Cfg::kStageBytes;
                    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    tma_load_4d(dst, &tm_a, bar, ks * Cfg::kSliceK, bm * Cfg::kTileM, 0, 0);
                    if (!B_NMAJOR) {
                        tma_load_4d(dst + Cfg::kABytes, &tm_b, bar, ks * Cfg::kSliceK, bn * Cfg::kTileN, 0, 0);
                    } else {
                        for (int x = 0; x < Cfg::kTileN / 64; ++x)  // boxes of 64 columns of B x 64 rows of K
                            tma_load_4d(dst + Cfg::kABytes + x * (Cfg::kSliceK * 128), &tm_b, bar,
                                        bn * Cfg::kTileN + x * 64, ks * Cfg::kSliceK, 0, 0);
                    }
                }
            }
        }
        if (!ok) {
            // abandoned: give the loads still in flight a bounded chance to land
            for (int it = max(0, ring - NS); it < ring; ++it)
                for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_full[it % NS]), (it / NS) & 1); ++w) {}
        }
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        const bool leader = elect_one();
        constexpr uint32_t idesc = make_idesc_bf16(Cfg::kTileM, Cfg::kTileN, B_NMAJOR ? 1 : 0);
        constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);
        constexpr uint32_t hi = uint32_t(desc_kmajor >> 32), lo = uint32_t(desc_kmajor);
        // N-contiguous B: 64-wide column groups are one box (64 K-rows x 128 B) apart, 8 K-rows 1024 B apart;
        // 16 K-rows further is 16 x 128 B
        constexpr uint64_t desc_nmajor = make_sdesc_sw128(Cfg::kSliceK * 128, 1024);
        constexpr uint32_t hi_b = B_NMAJOR ? uint32_t(desc_nmajor >> 32) : hi;
        constexpr uint32_t lo_b = B_NMAJOR ? uint32_t(desc_nmajor) : lo;
        constexpr uint32_t b_kstep = B_NMAJOR ? ((16 * 128) >> 4) : (32 >> 4);
        bool ok = true;
        int ring = 0;
        int n_done = 0;  // tiles this CTA has issued so far
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++n_done) {
            const int acc = n_done & 1;
            if (n_done >= 2) {  // the epilogue must have read this accumulator's previous tile out of TMEM
                ok = wait_bar(&bar_acc_empty[acc], ((n_done >> 1) - 1) & 1, STATUS_TIMEOUT_SOFTMAX);
                if (!ok) break;
            }
            const uint32_t d_tmem = tmem + acc * Cfg::kTileN;
            for (int ks = 0; ks < n_slices && ok; ++ks, ++ring) {
                const int slot = ring % NS;
                ok = wait_bar(&bar_full[slot], (ring / NS) & 1, STATUS_TIMEOUT_LOAD);
                if (!ok) break;
                tc_fence_after();
                if (leader) {
                    const uint32_t a_lo = lo | ((sRing + slot * Cfg::kStageBytes) >> 4);
                    const uint32_t b_lo = lo_b | ((sRing + slot * Cfg::kStageBytes + Cfg::kABytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < Cfg::kSliceK / 16; ++kk)
                        umma_ss_words(d_tmem, a_lo + ((kk * 32) >> 4), hi, b_lo + kk * b_kstep, hi_b, idesc,
                                      (ks > 0 || kk > 0));
                    umma_commit(smem_u32(&bar_empty[slot]));
                    if (ks == n_slices - 1) umma_commit(smem_u32(&bar_acc_full[acc]));
                }
            }
        }
        if (!ok) {  // abandoned: let the MMAs already issued finish before TMEM is released
            if (leader) umma_commit(smem_u32(&bar_drain));
            for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_drain), 0); ++w) {}
        }
    } else if (warp >= 4) {
        // =============================== epilogue ===============================
        const int wq = warp & 3;  // TMEM lane quadrant of this warp
        const uint32_t lane_sel = uint32_t(wq * 32) << 16;
        const uint32_t sC = sStage + wq * (Cfg::kOutBoxRows * 128);  // this warp's 32 staging rows
        bool ok = true;
        bool store_pending = false;  // (lane 0) a TMA store may still be reading this warp's staging rows
        int n_done = 0;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++n_done) {
            int bm, bn;
            gemm_tile_coords(tile, p, bm, bn);
            const int acc = n_done & 1;
            ok = wait_bar(&bar_acc_full[acc], (n_done >> 1) & 1, STATUS_TIMEOUT_MMA);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_acc = tmem + acc * Cfg::kTileN + lane_sel;
            const int row0 = bm * Cfg::kTileM + wq * 32;
#pragma unroll 1
            for (int c = 0; c < Cfg::kTileN / 32; ++c) {  // 32 columns at a time; two of them fill a 64-column box
                uint32_t v[32];
                tmem_ld_x32(t_acc + c * 32, v);
                tmem_wait_ld();
                if (c == Cfg::kTileN / 32 - 1) {  // the accumulator is in registers: the MMA warp may reuse it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                }
                if ((c & 1) == 0) {
                    // this warp's previous TMA store must have finished reading the staging rows
                    if (lane == 0 && store_pending) tma_store_wait_read();
                    __syncwarp();
                }
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint4 v4;
                    v4.x = pack_bf16x2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                    v4.y = pack_bf16x2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                    v4.z = pack_bf16x2(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5]));
                    v4.w = pack_bf16x2(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7]));
                    // 16-byte chunk `ch` of row `lane`, in the 128-byte-swizzled layout TMA expects
                    const int ch = (c & 1) * 4 + (e >> 3);
                    const uint32_t addr = sC + lane * 128 + ((ch ^ (lane & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v4.x), "r"(v4.y), "r"(v4.z),
                                 "r"(v4.w) : "memory");
                }
                if (c & 1) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    const int col0 = bn * Cfg::kTileN + (c >> 1) * 64;
                    if (lane == 0 && row0 < p.M && col0 < p.N) {
                        tma_store_4d(&tm_c, sC, col0, row0, 0, 0);
                        tma_store_commit();
                        store_pending = true;
                    }
                }
            }
        }
        if (lane == 0 && store_pending) tma_store_wait_all();
    }

    // ---- common exit: every thread arrives, then TMEM is released
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace ave
