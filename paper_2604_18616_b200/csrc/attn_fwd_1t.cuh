// Attention forward, single-sub-tile variant of the persistent warp-specialised kernel: a work tile
// is 128 query rows of one (batch, head), a CTA has one softmax warpgroup, and TWO CTAs share an SM.
//
// The two-sub-tile kernel (attn_fwd_ws.cuh) interleaves two 128-row sub-tiles inside one CTA so that
// the tensor pipe runs one sub-tile's products while the other's softmax is computed; its MMA warp
// serves both sub-tiles in a fixed order, and its K/V ring is shared, so the sub-tiles walk a tile in
// lock-step.  With few key steps per tile (short causal sequences: a 256-row tile of a 2048-token
// sequence has nine steps on average) the lock-step costs more than the sharing saves: sub-tile 0
// finishes a causal tile one step early and then waits for sub-tile 1 at every tile boundary.  Here the
// two chains of an SM are two independent CTAs, each with its own tile sequence, Q, K/V ring, TMEM half
// and MMA warp; one CTA's tile boundary (epilogue, next Q, pipeline refill) overlaps the other's steady
// state.  The price is that each CTA loads K and V for 128 rows instead of 256, i.e. twice the L2 and
// shared-memory traffic per query row; the launch code picks this kernel only where tiles are short.
//
//   warp 0        producer: TMA loads of Q and of the K/V ring
//   warp 1        MMA issuer: S = Q K_j^T and O += P V_j on tcgen05
//   warp 2        TMEM allocation / release and tile scheduler (cluster launch control)
//   warp 3        idle (register reallocation works on whole warpgroups of four warps)
//   warps 4..7    softmax + epilogue (one thread per query row)
//
// TMEM columns (256 per CTA): S [0,128), O [128,128+D); P (bf16 pairs) overwrites the first 64
// columns of S once a thread holds its whole score row in registers.
//
// The same kernel serves head dimensions above 128 (instantiated for D = 256; 136..248 run it on tensor maps
// of the true width, zero-filled): O then needs 256 TMEM columns, so a second sub-tile has no room, the CTA
// allocates all 512 columns and, with 64 KB each for the Q, K and V tiles, has an SM to itself.
#pragma once

#include <type_traits>

#include "attn_common.cuh"
#include "attn_fwd_ws.cuh"
#include "softmax_math.cuh"

namespace ave {

template <int D>
struct OneCfg {
    static constexpr int kThreads = 256;
    static constexpr int kTileBytes = BM * D * 2;            // the Q tile, a K tile or a V tile
    static constexpr int kBoxBytes = BM * 64 * 2;            // one 64-column TMA box (128 rows x 128 B)
    static constexpr int kBoxes = D / 64;
    static constexpr int kStages = (D >= 128) ? 2 : 4;       // ring slots, K and V tiles alternate (two CTAs must fit an SM)
    static constexpr int kSmemBytes = kTileBytes * (1 + kStages) + 1024;
    static constexpr int kCtasPerSm = (D <= 128) ? 2 : 1;
    static_assert(kCtasPerSm * (kSmemBytes + 2048) <= 228 * 1024, "the CTAs do not fit the shared memory of an SM");
    static constexpr uint32_t kTmemCols = (D <= 128) ? 256 : 512;
    static_assert(128 + D <= int(kTmemCols), "S and O do not fit the TMEM allocation");
    static constexpr uint32_t kColS = 0, kColO = 128;
    static constexpr int kRegsLight = 48;                    // producer / MMA / scheduler warpgroup
    static constexpr int kRegsSoftmax = 208;                 // softmax warpgroup
    // Two CTAs per SM: 65536 / (2 x 256) = 128 registers per thread at launch; setmaxnreg only moves registers
    // inside that allocation (the build and the launch code check the compiled image against it).
    static constexpr int kRegsAtLaunch = 128;
    static_assert(128 * kRegsLight + 128 * kRegsSoftmax <= kThreads * kRegsAtLaunch,
                  "register split exceeds the CTA's allocation");
    static constexpr int kTileConsumers = 6;                 // producer + MMA + 4 softmax warps read each tile
};

template <int D, bool CAUSAL, bool SPLIT, bool VARLEN = false>
__global__ void __launch_bounds__(256, 2)
attn_fwd_1t_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    if (threadIdx.x == 0) span_stamp(0);
    using Cfg = OneCfg<D>;
    using Tile = TileOf<SPLIT, VARLEN>;
    constexpr int NS = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(16) unsigned long long clc_response[2][2];
    __shared__ __align__(8) uint64_t bar_q_full, bar_q_empty, bar_s, bar_p, bar_o, bar_o_free;
    __shared__ __align__(8) uint64_t bar_full[NS], bar_empty[NS];
    __shared__ __align__(8) uint64_t bar_tile_full[2], bar_tile_ready[2], bar_tile_empty[2], bar_drain;
    __shared__ int tile_id[2];
    __shared__ Tile tile_info[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sRing = sQ + Cfg::kTileBytes;

    if (tid == 0) {
        abort_flag = (*reinterpret_cast<volatile unsigned int *>(&g_device_status) != 0) ? 1 : 0;
        mbar_init(smem_u32(&bar_q_full), 1);
        mbar_init(smem_u32(&bar_q_empty), 1);
        mbar_init(smem_u32(&bar_s), 1);
        mbar_init(smem_u32(&bar_p), 4);       // one arrival per softmax warp
        mbar_init(smem_u32(&bar_o), 1);
        mbar_init(smem_u32(&bar_o_free), 4);  // one arrival per softmax warp
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar_tile_full[t]), 1);
            mbar_init(smem_u32(&bar_tile_ready[t]), 1);
            mbar_init(smem_u32(&bar_tile_empty[t]), Cfg::kTileConsumers);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
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
    // The tile after a warp's n-th one (-1: none left), decoded by the scheduler warp.
    auto next_tile = [&](int n, bool &ok, Tile &w_out) -> int {
        const int slot = n & 1;
        ok = wait_bar(&bar_tile_ready[slot], (n >> 1) & 1, STATUS_TIMEOUT_SLOT);
        if (!ok) return -1;
        const int id = tile_id[slot];
        if (id >= 0) w_out = tile_info[slot];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_tile_empty[slot]));
        return id;
    };

    if (poisoned) {
        // nothing: fall through to the common exit
    } else if (warp < 4) {
        setmaxnreg_dec<Cfg::kRegsLight>();
        if (warp == 3) {
            // idle
        } else if (warp == 2) {
            // =============================== tile scheduler ===============================
            const bool leader = elect_one();
            bool ok = true;
            int last_id = blockIdx.x;   // the newest tile this CTA holds
            for (int k = 0; ok; ++k) {
                const int slot = k & 1;
                if (k >= 2) {  // every consumer has read the tile this slot held two requests ago
                    ok = wait_bar(&bar_tile_empty[slot], ((k >> 1) - 1) & 1, STATUS_TIMEOUT_SLOT);
                    if (!ok) break;
                }
                // over the launch's last tiles requests run one tile ahead, not two (see the two-sub-tile kernel)
                if (k >= 1 && p.total_blocks - last_id <= kLastWaves * Cfg::kCtasPerSm * int(n_sm())) {
                    ok = wait_bar(&bar_tile_empty[slot ^ 1], ((k - 1) >> 1) & 1, STATUS_TIMEOUT_SLOT);
                    if (!ok) break;
                }
                if (leader) {
                    mbar_arrive_expect_tx(smem_u32(&bar_tile_full[slot]), 16);
                    clc_try_cancel(smem_u32(&clc_response[slot][0]), smem_u32(&bar_tile_full[slot]));
                }
                ok = wait_bar(&bar_tile_full[slot], (k >> 1) & 1, STATUS_TIMEOUT_SLOT);
                if (!ok) break;
                const int id = clc_decode(clc_response[slot]);
                fence_proxy_async_smem();  // order the read before the slot's next asynchronous write
                if (id >= 0) {
                    const Tile w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
                    if (lane == 0) tile_info[slot] = w;
                }
                if (lane == 0) tile_id[slot] = id;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_tile_ready[slot]));
                if (id < 0) break;  // nothing left to take over: never ask again
                last_id = id;
            }
        } else if (warp == 0) {
            // =============================== producer ===============================
            const bool leader = elect_one();
            if (leader) {
                tma_prefetch_desc(&tm_q);
                tma_prefetch_desc(&tm_k);
                tma_prefetch_desc(&tm_v);
            }
            int ring = 0;  // K/V tiles loaded so far (ring position)
            bool ok = true;
            int id = blockIdx.x;
            Tile w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
            int q_tile = -1;  // number of the tile whose Q was loaded last
            for (int n = 0; id >= 0 && ok; ++n) {
                int id_next = -2;  // -2: not known yet
                Tile w_next = w;
                // Q of tile number tn (this tile or the next) goes in as soon as the tile before it has issued its
                // last Q K^T; the K/V loads must not queue behind it, so it is retried between them.
                auto try_load_q = [&](int tn, const Tile &wt, bool blocking) {
                    if (q_tile != tn - 1) return;
                    if (tn > 0) {
                        if (blocking) {
                            ok = wait_bar(&bar_q_empty, (tn - 1) & 1, STATUS_TIMEOUT_SLOT);
                            if (!ok) return;
                        } else if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&bar_q_empty), (tn - 1) & 1))) {
                            return;
                        }
                    }
                    q_tile = tn;
                    if (leader) {
                        const uint32_t bar = smem_u32(&bar_q_full);
                        mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                        for (int x = 0; x < Cfg::kBoxes; ++x)  // the tensor maps are {D, rows, heads, batch}
                            tma_load_4d(sQ + x * Cfg::kBoxBytes, &tm_q, bar, x * 64, q_base_of(wt) + wt.q0, wt.h,
                                        batch_coord(wt));
                    }
                };
                bool near_end = w.n0 <= 2;
                auto poll_q = [&]() {
                    try_load_q(n, w, false);
                    if (!near_end) return;
                    if (id_next == -2 &&
                        __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&bar_tile_ready[n & 1]), (n >> 1) & 1)))
                        id_next = next_tile(n, ok, w_next);  // does not wait: the phase has completed
                    if (id_next >= 0) try_load_q(n + 1, w_next, false);
                };
                poll_q();
                for (int it = 0; it < 2 * w.n0 && ok; ++it, ++ring) {  // it even: K_{it/2}; odd: V_{it/2}
                    const int slot = ring % NS, round = ring / NS;
                    near_end = it + 4 >= 2 * w.n0;
                    if (round > 0) {
                        const long long t0 = clock64();
                        for (;;) {
                            poll_q();
                            if (!ok) break;
                            if (__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&bar_empty[slot]), (round - 1) & 1))) break;
                            if (*reinterpret_cast<volatile int *>(&abort_flag) != 0) {
                                ok = false;
                                break;
                            }
                            if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                                abort_flag = 1;
                                atomicOr(&g_device_status, STATUS_TIMEOUT_SLOT);
                                ok = false;
                                break;
                            }
                            __nanosleep(40);
                        }
                        if (!ok) break;
                    } else {
                        poll_q();
                    }
                    if (leader) {
                        const uint32_t bar = smem_u32(&bar_full[slot]);
                        const CUtensorMap *tm = (it & 1) ? &tm_v : &tm_k;
                        mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                        for (int x = 0; x < Cfg::kBoxes; ++x)
                            tma_load_4d(sRing + slot * Cfg::kTileBytes + x * Cfg::kBoxBytes, tm, bar, x * 64,
                                        k_base_of(w) + key_begin(w) + (it >> 1) * BN, w.g, batch_coord(w));
                    }
                }
                if (ok) try_load_q(n, w, true);
                if (ok && id_next == -2) id_next = next_tile(n, ok, w_next);
                id = id_next;
                w = w_next;
            }
            if (!ok) {
                // abandoned: give the loads still in flight a bounded chance to land
                for (int it = max(0, ring - NS); it < ring; ++it)
                    for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_full[it % NS]), (it / NS) & 1); ++w) {}
            }
        } else {
            // =============================== MMA issuer ===============================
            const bool leader = elect_one();
            const uint32_t idesc_qk = make_idesc_bf16(BM, BN, 0) | ((p.scale_log2 < 0.f) ? (1u << 13) : 0u);
            constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, 1);
            constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);
            constexpr uint64_t desc_v = make_sdesc_sw128(BN * 128, 1024);
            const uint32_t tS = tmem + Cfg::kColS, tO = tmem + Cfg::kColO;
            bool ok = true;
            int ring = 0;      // ring position of the current tile's K_0
            uint32_t np = 0;   // P hand-offs taken so far (phase of bar_p)

            auto wait_full = [&](int idx) { return wait_bar(&bar_full[idx % NS], (idx / NS) & 1, STATUS_TIMEOUT_LOAD); };
            auto slot_addr = [&](int idx) { return sRing + (idx % NS) * Cfg::kTileBytes; };
            constexpr uint32_t hi_k = uint32_t(desc_kmajor >> 32), lo_k = uint32_t(desc_kmajor);
            constexpr uint32_t hi_v = uint32_t(desc_v >> 32), lo_v = uint32_t(desc_v);
            const uint32_t q_lo = lo_k | (sQ >> 4);
            auto issue_qk = [&](uint32_t k_addr) {
                if (leader) {
                    const uint32_t k_lo = lo_k | (k_addr >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t koff = ((kk / 4) * Cfg::kBoxBytes + (kk % 4) * 32) >> 4;
                        umma_ss_words(tS, q_lo + koff, hi_k, k_lo + koff, hi_k, idesc_qk, kk > 0);
                    }
                    umma_commit(smem_u32(&bar_s));
                }
            };
            auto issue_pv = [&](uint32_t v_addr, bool first) {
                if (leader) {
                    const uint32_t v_lo = lo_v | (v_addr >> 4);
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma_ts_words(tO, tS + kk * 8, v_lo + ((kk * 16 * 128) >> 4), hi_v, idesc_pv, (!first || kk > 0));
                }
            };
            // First step of tile number `tn` (tile `wt`, whose K_0 sits at ring position `ring0`): S = Q K_0^T,
            // issued right after the last P V of the tile before, so the pipeline does not drain at a tile boundary.
            auto start_tile = [&](const Tile &wt, int tn, int ring0) {
                ok = wait_bar(&bar_q_full, tn & 1, STATUS_TIMEOUT_LOAD);
                if (ok && wt.n0 > 0) ok = wait_full(ring0);
                if (!ok) return;
                if (wt.n0 > 0) {
                    tc_fence_after();
                    issue_qk(slot_addr(ring0));
                    if (leader) umma_commit(smem_u32(&bar_empty[ring0 % NS]));
                }
                if (leader && wt.n0 <= 1) umma_commit(smem_u32(&bar_q_empty));  // Q is released after its last Q K^T
            };

            int id = blockIdx.x;
            Tile w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
            start_tile(w, 0, 0);
            for (int n = 0; id >= 0 && ok; ++n) {
                const int nk = w.n0;
                Tile w_next = w;
                const int id_next = next_tile(n, ok, w_next);
                if (!ok) break;
                const int ring_next = ring + 2 * nk;
                if (id_next >= 0 && nk == 0) start_tile(w_next, n + 1, ring_next);  // nothing to do in this tile
                for (int j = 0; j < nk && ok; ++j) {
                    const int iv = ring + 2 * j + 1, ik = ring + 2 * j + 2;  // ring positions of V_j and K_{j+1}
                    ok = wait_full(iv);
                    if (ok && j + 1 < nk) ok = wait_full(ik);
                    // the previous tile's epilogue must have read O out of TMEM
                    if (ok && j == 0 && n > 0) ok = wait_bar(&bar_o_free, (n - 1) & 1, STATUS_TIMEOUT_SOFTMAX);
                    if (ok) ok = wait_bar(&bar_p, np & 1, STATUS_TIMEOUT_SOFTMAX);
                    if (!ok) break;
                    ++np;
                    tc_fence_after();
                    issue_pv(slot_addr(iv), j == 0);
                    if (leader) umma_commit(smem_u32(&bar_empty[iv % NS]));
                    if (leader && j == nk - 1) umma_commit(smem_u32(&bar_o));
                    if (j + 1 < nk) {
                        issue_qk(slot_addr(ik));
                        if (leader) umma_commit(smem_u32(&bar_empty[ik % NS]));
                        if (leader && j + 2 == nk) umma_commit(smem_u32(&bar_q_empty));
                    } else if (id_next >= 0) {
                        start_tile(w_next, n + 1, ring_next);
                        if (!ok) break;
                    }
                }
                ring = ring_next;
                id = id_next;
                w = w_next;
            }
            if (!ok) {  // abandoned: let the MMAs already issued finish before TMEM is released
                if (leader) umma_commit(smem_u32(&bar_drain));
                for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_drain), 0); ++w) {}
            }
        }
    } else {
        // =============================== softmax warpgroup ===============================
        setmaxnreg_inc<Cfg::kRegsSoftmax>();
        const int wq = warp & 3;                      // TMEM lane quadrant of this warp
        const int r = wq * 32 + lane;                 // row within the tile = TMEM lane
        const uint32_t lane_sel = uint32_t(wq * 32) << 16;
        const uint32_t tS = tmem + Cfg::kColS + lane_sel;
        const uint32_t tO = tmem + Cfg::kColO + lane_sel;
        // positive scale only; a negative one is applied by the tensor pipe, a zero one stands in as 2^-100
        // (see the two-sub-tile kernel)
        const float sl2 = (p.scale_log2 == 0.f) ? 7.888609052210118e-31f : fabsf(p.scale_log2);
        uint32_t ns = 0;             // S tiles consumed so far (phase of bar_s)
        uint32_t n_out = 0;          // finished O accumulators taken so far (phase of bar_o)
        bool ok = true;

        int id = blockIdx.x;
        Tile w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
        for (int n = 0; id >= 0 && ok; ++n) {
            const int bh = w.bh;
            const int sq = seq_q(w, p);                // query rows of this tile's sequence
            const int off = SPLIT ? p.causal_off : seq_k(w, p) - sq;
            const int i0 = w.q0;
            const int i = i0 + r;                     // query row
            const int n_t = w.n0;

            if (n_t == 0) {
                // no key visible to any row of this tile: O = 0, LSE = -inf
                if (i < sq) {
                    const uint4 z = make_uint4(0, 0, 0, 0);
                    if (SPLIT) {
                        const size_t row = (size_t(split_of(w)) * p.BH + bh) * p.Sq + i;
                        for (int c = 0; c < D / 4; ++c) reinterpret_cast<uint4 *>(p.o_partial + row * D)[c] = z;
                        p.lse_partial[row] = -INFINITY;
                    } else {
                        __nv_bfloat16 *o_row = reinterpret_cast<__nv_bfloat16 *>(p.o) + batch_coord(w) * p.o_stride_b +
                                               w.h * p.o_stride_h + (q_base_of(w) + i) * p.o_stride_r;
                        for (int c = 0; c < p.d_true / 8; ++c) reinterpret_cast<uint4 *>(o_row)[c] = z;
                        p.lse[lse_index(w, p, i)] = -INFINITY;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_o_free));  // O was not used: hand it back at once
            } else {
                float m_run = -INFINITY, l_run = 0.f;
                const int k_end = key_end(w, p);
                const int n_full = unmasked_steps<CAUSAL, SPLIT>(i0, n_t, key_begin(w), k_end, off, p.rows_per_head);
                auto step = [&](const int j, auto masked) -> bool {
                    // `masked` is a run-time bool (causal kernels) or std::true_type / std::false_type
                    constexpr bool kRuntimeFlag = std::is_same<decltype(masked), bool>::value;
                    bool need_mask;
                    if constexpr (kRuntimeFlag) need_mask = masked;
                    else need_mask = decltype(masked)::value;
                    ok = wait_bar(&bar_s, ns & 1, STATUS_TIMEOUT_MMA);
                    if (!ok) return false;
                    ++ns;
                    tc_fence_after();
                    uint32_t sraw[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld_x32(tS + c * 32, sraw[c]);
                    tmem_wait_ld();
                    const int mask_trips = kRuntimeFlag ? opaque(need_mask ? 1 : 0) : int(need_mask);
#pragma unroll 1
                    for (int trip = 0; trip < mask_trips; ++trip) {
                        const int j0 = key_begin(w) + j * BN;  // first key of this step
                        int lim = k_end - 1 - j0;               // columns c <= lim of this tile are visible to row i
                        if constexpr (SPLIT) {
                            const int pos = p.rows_per_head > 0 ? i % p.rows_per_head : i;  // query position of row i
                            if (CAUSAL) lim = min(lim, pos + off - j0);
                        } else {
                            if (CAUSAL) lim = min(lim, i + off - j0);
                        }
                        // a masked score becomes -inf: it drops out of the maximum and its probability is exactly 0
#pragma unroll
                        for (int c = 0; c < 128; ++c)
                            sraw[c >> 5][c & 31] = (c <= lim) ? sraw[c >> 5][c & 31] : 0xff800000u;
                    }
                    // row maximum of the (masked) raw scores, as scale*log2(e)*s; -inf if nothing is visible
                    float m_tile;
                    {
                        float e0 = -INFINITY, e1 = -INFINITY, e2 = -INFINITY, e3 = -INFINITY;
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            e0 = max3(e0, __uint_as_float(sraw[0][c]), __uint_as_float(sraw[0][c + 1]));
                            e1 = max3(e1, __uint_as_float(sraw[1][c]), __uint_as_float(sraw[1][c + 1]));
                            e2 = max3(e2, __uint_as_float(sraw[2][c]), __uint_as_float(sraw[2][c + 1]));
                            e3 = max3(e3, __uint_as_float(sraw[3][c]), __uint_as_float(sraw[3][c + 1]));
                        }
                        const float ext = fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
                        m_tile = (ext == -INFINITY) ? -INFINITY : ext * sl2;
                    }
                    // running maximum, moved lazily (see kRescaleThreshold)
                    float alpha = 1.f;
                    if (j == 0) {
                        m_run = m_tile;
                    } else if (m_tile - m_run > rescale_margin(l_run)) {
                        alpha = ex2_approx(m_run - m_tile);
                        m_run = m_tile;
                    }
                    // p = exp2(scale*log2e*s - m) for the whole row: P -> bf16 pairs into TMEM over the first 64
                    // columns of S; the row sum is taken from the fp32 probabilities, before the rounding
                    {
                        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
                        float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                        const float2 sc2 = make_float2(sl2, sl2), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            uint32_t pk[16];
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                const float2 x = __ffma2_rn(
                                    make_float2(__uint_as_float(sraw[cc][e]), __uint_as_float(sraw[cc][e + 1])), sc2, nm2);
                                float2 pr;
                                if ((kFmaPipeExpMask >> ((e >> 1) & 7)) & 1) {
                                    pr = exp2_fma_pipe(x);
                                } else {
                                    pr.x = ex2_approx(x.x);
                                    pr.y = ex2_approx(x.y);
                                }
                                if (e & 2) acc1 = __fadd2_rn(acc1, pr);
                                else       acc0 = __fadd2_rn(acc0, pr);
                                pk[e >> 1] = pack_bf16x2(pr.x, pr.y);
                            }
                            tmem_st_x16(tS + cc * 16, pk);
                        }
                        // O <- alpha * O, after the exponentiation: the score registers are free by then, so the whole
                        // accumulator row (128 columns at a time) is in flight at once.  S(j) ready implies P V_{j-1} has
                        // finished (in-order tensor pipe), and P V_j is not issued before this thread's arrival below.
                        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                            constexpr int kGroup = (D < 128) ? D : 128;
#pragma unroll 1
                            for (int g = 0; g < D; g += kGroup) {
                                uint32_t oc[kGroup / 32][32];
#pragma unroll
                                for (int c = 0; c < kGroup / 32; ++c) tmem_ld_x32(tO + g + c * 32, oc[c]);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < kGroup / 32; ++c) {
#pragma unroll
                                    for (int e = 0; e < 32; ++e) oc[c][e] = __float_as_uint(__uint_as_float(oc[c][e]) * alpha);
                                    tmem_st_x32(tO + g + c * 32, oc[c]);
                                }
                            }
                        }
                        l_run = l_run * alpha + ((acc0.x + acc0.y) + (acc1.x + acc1.y));
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_p));
                    return true;
                };
                {
                    if constexpr (CAUSAL) {
                        for (int j = 0; j < n_t; ++j)
                            if (!step(j, j >= n_full)) break;
                    } else {
                        // only a ragged last key tile is masked here: a copy of the step for it costs nothing
                        int j = 0;
                        for (; j < n_full; ++j)
                            if (!step(j, std::false_type{})) break;
                        for (; ok && j < n_t; ++j)
                            if (!step(j, std::true_type{})) break;
                    }
                }

                // ---- epilogue: O / l -> bf16 -> global (each thread its own row); LSE = ln2 * (m + log2 l)
                if (ok) ok = wait_bar(&bar_o, n_out & 1, STATUS_TIMEOUT_MMA);
                if (ok) {
                    ++n_out;
                    tc_fence_after();
                    const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
                    const float lse_row = (l_run > 0.f) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                    const size_t prow = SPLIT ? (size_t(split_of(w)) * p.BH + bh) * p.Sq + i : 0;
                    __nv_bfloat16 *o_row = reinterpret_cast<__nv_bfloat16 *>(p.o) + batch_coord(w) * p.o_stride_b +
                                           w.h * p.o_stride_h + (q_base_of(w) + i) * p.o_stride_r;
                    if (SPLIT) {
                        if (i < p.Sq) p.lse_partial[prow] = lse_row;
                    } else {
                        if (i < sq) p.lse[lse_index(w, p, i)] = lse_row;
                    }
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t oc[32];
                        tmem_ld_x32(tO + c * 32, oc);
                        tmem_wait_ld();
                        if (c == D / 32 - 1) {  // O is in registers: the next tile may overwrite it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(smem_u32(&bar_o_free));
                        }
                        if (SPLIT) {
                            // partial result of this key range: normalised O in fp32, straight to global
                            if (i < p.Sq) {
#pragma unroll
                                for (int e = 0; e < 32; e += 4)
                                    reinterpret_cast<float4 *>(p.o_partial + prow * D + c * 32)[e >> 2] =
                                        make_float4(__uint_as_float(oc[e]) * inv_l, __uint_as_float(oc[e + 1]) * inv_l,
                                                    __uint_as_float(oc[e + 2]) * inv_l, __uint_as_float(oc[e + 3]) * inv_l);
                            }
                        } else if (i < sq) {
#pragma unroll
                            for (int e = 0; e < 32; e += 8) {
                                uint4 v4;
                                v4.x = pack_bf16x2(__uint_as_float(oc[e]) * inv_l, __uint_as_float(oc[e + 1]) * inv_l);
                                v4.y = pack_bf16x2(__uint_as_float(oc[e + 2]) * inv_l, __uint_as_float(oc[e + 3]) * inv_l);
                                v4.z = pack_bf16x2(__uint_as_float(oc[e + 4]) * inv_l, __uint_as_float(oc[e + 5]) * inv_l);
                                v4.w = pack_bf16x2(__uint_as_float(oc[e + 6]) * inv_l, __uint_as_float(oc[e + 7]) * inv_l);
                                if (c * 32 + e < p.d_true) *reinterpret_cast<uint4 *>(o_row + c * 32 + e) = v4;
                            }
                        }
                    }
                }
            }
            if (ok) id = next_tile(n, ok, w);
        }
    }

    // ---- common exit: every thread arrives, then TMEM is released
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, Cfg::kTmemCols);
    if (threadIdx.x == 0) span_stamp(1);
}

}  // namespace ave
