// Attention forward, persistent warp-specialised kernel for sm_100a.
//
// A work tile is a block of 256 query rows of one (batch, head) - or, in causal
// launches with an even number of query heads per key/value head, the same 128
// query rows of two neighbouring heads: two 128-row
// sub-tiles that ping-pong so the tensor pipe works on one while the softmax
// of the other runs (the paper's "+Pipe": software pipelining across disjoint
// groups of warps, Section 9; steps of the loop as in Section 2 / Fig. 1).
// The grid has one CTA per work tile, ordered so that tiles sharing K/V run
// together and long causal tiles come first; a CTA that finishes its tile
// takes over a not-yet-started CTA's tile through cluster launch control, so
// the resident CTAs persist and prefetch their next tile while finishing the
// current one.
//
//   warp 0        producer: TMA loads of Q and of the K/V ring
//   warp 1        MMA issuer: S_t = Q_t K_j^T and O_t += P_t V_j on tcgen05
//   warp 2        TMEM allocation / release
//   warp 3        tile scheduler (cluster launch control)
//   warps 4..7    softmax + epilogue of sub-tile 0 (one thread per query row)
//   warps 8..11   softmax + epilogue of sub-tile 1
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [384,384+D); P_t
// (bf16 pairs) overwrites the first 64 columns of S_t once a thread holds its
// whole score row in registers.
#pragma once

#include <type_traits>

#include "attn_common.cuh"
#include "softmax_math.cuh"

namespace ave {

template <int D>
struct WsCfg {
    static constexpr int kThreads = 384;
    static constexpr int kQRows = 2 * BM;                    // query rows per work tile
    static constexpr int kTileBytes = BM * D * 2;            // one Q sub-tile, K tile or V tile
    static constexpr int kBoxBytes = BM * 64 * 2;            // one 64-column TMA box (128 rows x 128 B)
    static constexpr int kBoxes = D / 64;
    static constexpr int kStages = (D == 128) ? 4 : 8;       // ring slots, K and V tiles alternate
    static constexpr int kStageOBytes = kBoxBytes;           // O staging per sub-tile: 64 columns at a time
    static constexpr int kOutBoxRows = 32;                   // each softmax warp stores its own 32 rows
    static constexpr int kSmemBytes = kTileBytes * (2 + kStages) + 2 * kStageOBytes + 1024;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kRegsLight = 64;                    // producer / MMA / scheduler warpgroup
    static constexpr int kRegsSoftmax = 216;                 // softmax warpgroups
    // setmaxnreg only moves registers inside what the CTA was given at launch (kThreads x the
    // per-thread count ptxas reports, 168 for 384 threads); asking for more blocks forever.
    static constexpr int kRegsAtLaunch = 168;
    static_assert(128 * kRegsLight + 256 * kRegsSoftmax <= kThreads * kRegsAtLaunch,
                  "register split exceeds the CTA's allocation");
    static constexpr int kTileConsumers = 10;               // producer + MMA + 8 softmax warps read each tile id
};

// Over the last kLastWaves x (resident CTAs) tiles of a launch a CTA claims one tile ahead instead of two.
constexpr int kLastWaves = 2;

// Rescale O only when the running maximum moved by more than this many powers of two; until then
// probabilities are taken relative to a stale maximum (at most 2^32 too large), which the final division by l
// undoes.  The exponent range is no concern: P is rounded to bf16, which has fp32's range, and l and O stay
// below 2^32 * Sk * max|V|, far from fp32's limit ...
constexpr float kRescaleThreshold = 32.0f;
// ... unless the new maximum would outweigh the sum accumulated so far.  A probability taken relative to a
// stale maximum is an arbitrary number, rounded to bf16 with a relative error of up to 2^-9; for a key that
// dominates its row that error is the error of O (0.2 % of a |V| of 4 is 0.008: together with the rounding
// of O itself that is beyond the 2e-2 allowed, and the long-context configuration's peaked rows showed it).
// Relative to its own maximum the dominant probability is exactly 1.  So the maximum also moves when
// 2^(m_tile - m_run) exceeds l, the sum accumulated so far; terms that stay below half of a row's sum keep
// their rounding errors, which average out.  (Measured on the long-context configuration: every element
// then lies within the rounding of O itself, at +9 % time there and no change on unpeaked inputs.)
__device__ __forceinline__ float rescale_margin(float l_run) {
    return fminf(kRescaleThreshold, fmaxf(0.f, __log2f(l_run)));
}

// Of every 8 consecutive pairs of probabilities, the pairs whose bit is set
// here are exponentiated on the FMA pipe (exp2_fma_pipe) instead of the
// exponential unit.
#ifndef AVE_FMA_EXP_MASK
#define AVE_FMA_EXP_MASK 0x11  // 2 of 8: a quarter of the exponentials (more measured slower, fewer gains less)
#endif
constexpr unsigned kFmaPipeExpMask = AVE_FMA_EXP_MASK;

// Trace builds record the role timeline of two consecutive tiles of a CTA, starting at this one (0 = its first);
// the second tile's steps follow at iteration index 32 (steps beyond the 27th of a tile share its slot).
#ifndef AVE_TRACE_TILE
#define AVE_TRACE_TILE 0
#endif
constexpr int kTraceTile = AVE_TRACE_TILE;
__device__ __forceinline__ bool traced(int n) { return unsigned(n - kTraceTile) < 2u; }
__device__ __forceinline__ int trace_it(int n, int j) { return (n - kTraceTile) * 32 + (j < 28 ? j : 27); }  // 28, 30: per-tile stamps

template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// ---- cluster launch control: take over the tile of a CTA that has not started
__device__ __forceinline__ void clc_try_cancel(uint32_t response_smem, uint32_t bar) {
    asm volatile("clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
                 ::"r"(response_smem), "r"(bar) : "memory");
}
// Decode a 16-byte response: the cancelled CTA's blockIdx.x, or -1 if nothing was cancelled.
__device__ __forceinline__ int clc_decode(const volatile unsigned long long *response) {
    const unsigned long long lo = response[0], hi = response[1];
    uint32_t ok, x;
    asm volatile(
        "{\n"
        ".reg .b128 resp;\n"
        ".reg .pred p;\n"
        "mov.b128 resp, {%2, %3};\n"
        "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p, resp;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "mov.u32 %1, 0;\n"
        "@p clusterlaunchcontrol.query_cancel.get_first_ctaid::x.b32.b128 %1, resp;\n"
        "}\n"
        : "=r"(ok), "=r"(x)
        : "l"(lo), "l"(hi));
    return ok ? int(x) : -1;
}

template <int D, bool CAUSAL, bool SPLIT, bool VARLEN = false>
__global__ void __launch_bounds__(384, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                   const FwdParams p) {
    if (threadIdx.x == 0) span_stamp(0);
    using Cfg = WsCfg<D>;
    constexpr int NS = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(16) unsigned long long clc_response[2][2];
    __shared__ __align__(8) uint64_t bar_q_full[2], bar_q_empty[2], bar_s[2], bar_p[2], bar_o[2], bar_o_free[2];
    __shared__ __align__(8) uint64_t bar_full[NS], bar_empty[NS];
    __shared__ __align__(8) uint64_t bar_tile_full[2], bar_tile_ready[2], bar_tile_empty[2], bar_drain;
    // The scheduler warp decodes every tile it obtains once, for all warps: index and decoded form, two in flight.
    __shared__ int tile_id[2];
    __shared__ TileOf<SPLIT, VARLEN> tile_info[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;                                   // two sub-tiles
    const uint32_t sRing = sQ + 2 * Cfg::kTileBytes;                 // NS slots
    const uint32_t sStage = sRing + NS * Cfg::kTileBytes;            // O staging, one box per sub-tile

    if (tid == 0) {
        // A wait that ran out earlier (in this launch or a previous one) leaves the
        // status word set until the host reads it; later CTAs then skip their work
        // instead of each running into the same limit.
        abort_flag = (*reinterpret_cast<volatile unsigned int *>(&g_device_status) != 0) ? 1 : 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar_q_full[t]), 1);
            mbar_init(smem_u32(&bar_q_empty[t]), 1);
            mbar_init(smem_u32(&bar_s[t]), 1);
            mbar_init(smem_u32(&bar_p[t]), 4);       // one arrival per softmax warp
            mbar_init(smem_u32(&bar_o[t]), 1);
            mbar_init(smem_u32(&bar_o_free[t]), 4);  // one arrival per softmax warp
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

    // A full warp waits on an mbarrier phase; the verdict is made warp-uniform.
    auto wait_bar = [&](uint64_t *bar, uint32_t parity, unsigned code) -> bool {
        const bool r = mbar_wait_bounded(smem_u32(bar), parity, &abort_flag, code);
        return __all_sync(0xffffffffu, r);
    };
    // Every consumer warp of the tile sequence calls this to learn the tile after its n-th one (-1: none
    // left) and takes the decoded tile from shared memory; one lane releases the slot.
    auto next_tile = [&](int n, bool &ok, TileOf<SPLIT, VARLEN> &w_out) -> int {
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
            // =============================== tile scheduler ===============================
            const bool leader = elect_one();
            bool ok = true;
            int last_id = blockIdx.x;   // the newest tile this CTA holds
            for (int k = 0; ok; ++k) {
                const int slot = k & 1;
                if (k >= 2) {  // every consumer has read the response this slot held two requests ago
                    ok = wait_bar(&bar_tile_empty[slot], ((k >> 1) - 1) & 1, STATUS_TIMEOUT_SLOT);
                    if (!ok) break;
                }
                // Requests normally run two tiles ahead of the tile the CTA works on.  Over the launch's last
                // tiles they run one ahead only (request k waits until every warp has read response k-1,
                // that is, has begun the tile it named): a tile claimed early there is one that an SM about
                // to go idle could have taken.  With two ahead throughout, the last CTA of a 2048-token
                // causal launch ended 30 us after the median one; with one ahead throughout, the MMA warp
                // waits for its next tile at many tile ends.
                if (k >= 1 && p.total_blocks - last_id <= kLastWaves * int(n_sm())) {
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
                    const TileOf<SPLIT, VARLEN> w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
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
            TileOf<SPLIT, VARLEN> w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
            int q_tile[2] = {-1, -1};  // number of the tile whose Q_t was loaded last
            for (int n = 0; id >= 0 && ok; ++n) {
                if (traced(n) && leader) trace_stamp(3, (n - kTraceTile) * 32 + 28, 0);
                // The tile after this one, as soon as the scheduler warp has it: its Q_t can go in before this
                // tile's last K and V do (Q comes from HBM, the K/V of a launch group mostly from L2).
                int id_next = -2;  // -2: not known yet
                TileOf<SPLIT, VARLEN> w_next = w;
                // Q_t of tile number tn (this tile or the next) goes in as soon as the tile before it has issued
                // its last Q_t K^T.  Q_1 is released later than Q_0 (causal sub-tile 1 runs one step longer), and
                // the K/V tiles must not queue behind it, so a Q load that cannot go yet stays pending and is
                // retried between the K/V loads.
                auto try_load_q = [&](int t, int tn, const TileOf<SPLIT, VARLEN> &wt, bool blocking) {
                    if (q_tile[t] != tn - 1) return;  // loaded already, or the tile before it is not in yet
                    if (tn > 0) {
                        if (blocking) {
                            ok = wait_bar(&bar_q_empty[t], (tn - 1) & 1, STATUS_TIMEOUT_SLOT);
                            if (!ok) return;
                        } else if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&bar_q_empty[t]), (tn - 1) & 1))) {
                            return;
                        }
                    }
                    q_tile[t] = tn;
                    if (leader) {
                        if (traced(tn)) trace_stamp(3, (tn - kTraceTile) * 32 + 28, 1 + t);
                        const uint32_t bar = smem_u32(&bar_q_full[t]);
                        mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                        for (int x = 0; x < Cfg::kBoxes; ++x)  // the tensor maps are {D, rows, heads, batch}
                            tma_load_4d(sQ + t * Cfg::kTileBytes + x * Cfg::kBoxBytes, &tm_q, bar, x * 64,
                                        q_base_of(wt) + wt.q0 + t * wt.dq, wt.h + t * wt.dh, batch_coord(wt));
                    }
                };
                bool near_end = w.n1 <= 2;  // the next tile is looked for only while this tile's last loads wait for their slots
                auto poll_q = [&]() {
                    try_load_q(0, n, w, false);
                    try_load_q(1, n, w, false);
                    if (!near_end) return;
                    if (id_next == -2 &&
                        __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&bar_tile_ready[n & 1]), (n >> 1) & 1)))
                        id_next = next_tile(n, ok, w_next);  // does not wait: the phase has completed
                    if (id_next >= 0) {
                        try_load_q(0, n + 1, w_next, false);
                        try_load_q(1, n + 1, w_next, false);
                    }
                };
                poll_q();
                for (int it = 0; it < 2 * w.n1 && ok; ++it, ++ring) {  // it even: K_{it/2}; odd: V_{it/2}
                    const int slot = ring % NS, round = ring / NS;
                    near_end = it + 4 >= 2 * w.n1;
                    if (round > 0) {
                        // Poll for the slot without blocking: a Q buffer may free up first, and the MMA
                        // warp may be waiting for that Q before it releases any more slots.
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
                        if (traced(n)) trace_stamp(3, trace_it(n, it >> 1), it & 1);
                        mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                        for (int x = 0; x < Cfg::kBoxes; ++x)
                            tma_load_4d(sRing + slot * Cfg::kTileBytes + x * Cfg::kBoxBytes, tm, bar, x * 64,
                                        k_base_of(w) + key_begin(w) + (it >> 1) * BN, w.g, batch_coord(w));
                    }
                }
                if (ok) try_load_q(0, n, w, true);
                if (ok) try_load_q(1, n, w, true);
                if (traced(n) && leader) trace_stamp(3, (n - kTraceTile) * 32 + 28, 3);
                if (ok && id_next == -2) id_next = next_tile(n, ok, w_next);
                if (traced(n) && leader) trace_stamp(3, (n - kTraceTile) * 32 + 28, 4);
                id = id_next;
                w = w_next;
            }
            if (!ok) {
                // abandoned: give the loads still in flight a bounded chance to land
                for (int it = max(0, ring - NS); it < ring; ++it)
                    for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_full[it % NS]), (it / NS) & 1); ++w) {}
            }
        } else if (warp == 1) {
            // =============================== MMA issuer ===============================
            // The whole warp runs this loop so that addresses and descriptors stay
            // warp-uniform; one elected lane issues the tcgen05 instructions.
            const bool leader = elect_one();
            // A negative scale turns the row maximum of scale*s into the minimum of s; the softmax works
            // with |scale| on scores the tensor pipe has negated (bit 13 of the descriptor negates A).
            const uint32_t idesc_qk = make_idesc_bf16(BM, BN, 0) | ((p.scale_log2 < 0.f) ? (1u << 13) : 0u);
            constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, 1);
            constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);
            constexpr uint64_t desc_v = make_sdesc_sw128(BN * 128, 1024);
            const uint32_t tS[2] = {tmem + Cfg::kColS0, tmem + Cfg::kColS1};
            const uint32_t tO[2] = {tmem + Cfg::kColO0, tmem + Cfg::kColO1};
            bool ok = true;
            int ring = 0;             // ring position of the current tile's K_0
            uint32_t np[2] = {0, 0};  // P_t hand-offs taken so far (phase of bar_p[t])

            auto wait_full = [&](int idx) { return wait_bar(&bar_full[idx % NS], (idx / NS) & 1, STATUS_TIMEOUT_LOAD); };
            auto slot_addr = [&](int idx) { return sRing + (idx % NS) * Cfg::kTileBytes; };
            // Descriptors as (low, high) words: the high word is constant per operand kind, the low
            // word is the constant part plus address/16, so stepping along K is one 32-bit add.
            constexpr uint32_t hi_k = uint32_t(desc_kmajor >> 32), lo_k = uint32_t(desc_kmajor);
            constexpr uint32_t hi_v = uint32_t(desc_v >> 32), lo_v = uint32_t(desc_v);
            const uint32_t q_lo[2] = {lo_k | (sQ >> 4), lo_k | ((sQ + Cfg::kTileBytes) >> 4)};
            auto issue_qk = [&](int t, uint32_t k_addr) {
                if (leader) {
                    const uint32_t k_lo = lo_k | (k_addr >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t koff = ((kk / 4) * Cfg::kBoxBytes + (kk % 4) * 32) >> 4;
                        umma_ss_words(tS[t], q_lo[t] + koff, hi_k, k_lo + koff, hi_k, idesc_qk, kk > 0);
                    }
                    umma_commit(smem_u32(&bar_s[t]));
                }
            };
            auto issue_pv = [&](int t, uint32_t v_addr, bool first) {
                if (leader) {
                    const uint32_t v_lo = lo_v | (v_addr >> 4);
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma_ts_words(tO[t], tS[t] + kk * 8, v_lo + ((kk * 16 * 128) >> 4), hi_v, idesc_pv,
                                      (!first || kk > 0));
                }
            };

            // First step of sub-tile t in tile number `tn` (tile `wt`, whose K_0 sits at ring position
            // `ring0`): S_t = Q_t K_0^T.  Issued as soon as sub-tile t has finished the tile before, so
            // the next tile's first scores are computed while the other sub-tile is still at work.
            auto start_subtile = [&](int t, const TileOf<SPLIT, VARLEN> &wt, int tn, int ring0) {
                const int n_t = t ? wt.n1 : wt.n0;
                ok = wait_bar(&bar_q_full[t], tn & 1, STATUS_TIMEOUT_LOAD);
                if (ok && n_t > 0) ok = wait_full(ring0);
                if (!ok) return;
                if (n_t > 0) {
                    tc_fence_after();
                    issue_qk(t, slot_addr(ring0));
                }
                // sub-tile 1 always visits at least as many key tiles as sub-tile 0: it is the last user of K_0
                if (leader && t == 1 && wt.n1 > 0) umma_commit(smem_u32(&bar_empty[ring0 % NS]));
                // Q_t is released after the last Q_t K^T of the tile (here if there is at most one)
                if (leader && n_t <= 1) umma_commit(smem_u32(&bar_q_empty[t]));
            };

            int id = blockIdx.x;
            TileOf<SPLIT, VARLEN> w = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
            start_subtile(0, w, 0, 0);
            if (ok) start_subtile(1, w, 0, 0);
            for (int n = 0; id >= 0 && ok; ++n) {
                const int n0 = w.n0, n1 = w.n1;
                if (lane == 0) trace_stamp(3, n, 7);  // start of this CTA's n-th tile
                // the tile after this one (its first steps are issued from inside this tile's loop)
                TileOf<SPLIT, VARLEN> w_next = w;
                const int id_next = next_tile(n, ok, w_next);
                if (!ok) break;
                const int ring_next = ring + 2 * n1;
                if (id_next >= 0 && n1 == 0) {  // nothing to do in this tile at all
                    start_subtile(0, w_next, n + 1, ring_next);
                    if (ok) start_subtile(1, w_next, n + 1, ring_next);
                }
                for (int j = 0; j < n1 && ok; ++j) {
                    const int iv = ring + 2 * j + 1, ik = ring + 2 * j + 2;  // ring positions of V_j and K_{j+1}
                    if (traced(n) && lane == 0) trace_stamp(0, trace_it(n, j), 0);
                    // Everything this step needs from the ring and from the previous tile is checked
                    // first, while the softmax of this step is still running; after that only the two
                    // P hand-offs stand between this warp and the tensor pipe.
                    ok = wait_full(iv);
                    if (ok && j + 1 < n1) ok = wait_full(ik);
                    if (ok && j == 0 && n > 0) {  // the previous tile's epilogue must have read O_t out of TMEM
                        if (n0 > 0) ok = wait_bar(&bar_o_free[0], (n - 1) & 1, STATUS_TIMEOUT_SOFTMAX);
                        ok = ok && wait_bar(&bar_o_free[1], (n - 1) & 1, STATUS_TIMEOUT_SOFTMAX);
                    }
                    if (!ok) break;
                    const uint32_t v_addr = slot_addr(iv), k_addr = slot_addr(ik);
                    if (j < n0) {
                        ok = wait_bar(&bar_p[0], np[0] & 1, STATUS_TIMEOUT_SOFTMAX);
                        if (!ok) break;
                        ++np[0];
                        if (traced(n) && lane == 0) trace_stamp(0, trace_it(n, j), 1);
                        tc_fence_after();
                        issue_pv(0, v_addr, j == 0);
                        if (leader && j == n0 - 1) umma_commit(smem_u32(&bar_o[0]));
                        if (j + 1 < n0) {
                            issue_qk(0, k_addr);
                            if (leader && j + 2 == n0) umma_commit(smem_u32(&bar_q_empty[0]));
                        } else if (id_next >= 0) {
                            start_subtile(0, w_next, n + 1, ring_next);  // sub-tile 0 moves on to the next tile
                            if (!ok) break;
                        }
                    }
                    if (traced(n) && lane == 0) trace_stamp(0, trace_it(n, j), 2);
                    ok = wait_bar(&bar_p[1], np[1] & 1, STATUS_TIMEOUT_SOFTMAX);
                    if (!ok) break;
                    ++np[1];
                    if (traced(n) && lane == 0) trace_stamp(0, trace_it(n, j), 3);
                    tc_fence_after();
                    issue_pv(1, v_addr, j == 0);
                    if (leader) umma_commit(smem_u32(&bar_empty[iv % NS]));
                    if (leader && j == n1 - 1) umma_commit(smem_u32(&bar_o[1]));
                    if (j + 1 < n1) {
                        issue_qk(1, k_addr);
                        if (leader) umma_commit(smem_u32(&bar_empty[ik % NS]));
                        if (leader && j + 2 == n1) umma_commit(smem_u32(&bar_q_empty[1]));
                    } else if (id_next >= 0) {
                        if (n0 == 0) start_subtile(0, w_next, n + 1, ring_next);  // sub-tile 0 had nothing to do here
                        if (ok) start_subtile(1, w_next, n + 1, ring_next);
                        if (!ok) break;
                    }
                    if (traced(n) && lane == 0) trace_stamp(0, trace_it(n, j), 4);
                }
                ring = ring_next;
                id = id_next;
                w = w_next;
                if (lane == 0) span_stamp(2, n + 1);
            }
            if (!ok) {  // abandoned: let the MMAs already issued finish before TMEM is released
                if (leader) umma_commit(smem_u32(&bar_drain));
                for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_test_wait(smem_u32(&bar_drain), 0); ++w) {}
            }
        }
    } else {
        // =============================== softmax warpgroups ===============================
        setmaxnreg_inc<Cfg::kRegsSoftmax>();
        const int t = (warp - 4) >> 2;                // sub-tile
        const int wq = warp & 3;                      // TMEM lane quadrant of this warp
        const int r = wq * 32 + lane;                 // row within the sub-tile = TMEM lane
        const uint32_t lane_sel = uint32_t(wq * 32) << 16;
        const uint32_t tS = tmem + (t ? Cfg::kColS1 : Cfg::kColS0) + lane_sel;
        const uint32_t tO = tmem + (t ? Cfg::kColO1 : Cfg::kColO0) + lane_sel;
        const uint32_t sO = sStage + t * Cfg::kStageOBytes + wq * (Cfg::kOutBoxRows * 128);  // this warp's 32 rows
        // The softmax works with a positive scale only, which keeps one maximum-then-exponentiate
        // code path (the kernel's code has to stay within the instruction cache): for a negative scale
        // the MMA warp has the tensor pipe negate the scores and |scale| is used here; a zero scale
        // (all visible keys weigh the same) is replaced by 2^-100, under which every visible score
        // still rounds to an exponent of 0 while a masked one stays -inf.
        const float sl2 = (p.scale_log2 == 0.f) ? 7.888609052210118e-31f : fabsf(p.scale_log2);
        const bool tracer = (r == 0);
        uint32_t ns = 0;             // S_t tiles consumed so far (phase of bar_s[t])
        uint32_t n_out = 0;          // finished O_t accumulators taken so far (phase of bar_o[t])
        bool ok = true;
        bool store_pending = false;  // (lane 0) a TMA store may still be reading this warp's staging rows

        int id = blockIdx.x;
        TileOf<SPLIT, VARLEN> w_tile = decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
        for (int n = 0; id >= 0 && ok; ++n) {
            TileOf<SPLIT, VARLEN> w = w_tile;
            w.h += t * w.dh;                           // this sub-tile's query head (head-paired launches)
            w.bh += t * w.dh;
            const int bh = w.bh;
            const int sq = seq_q(w, p);                // query rows of this tile's sequence
            const int off = SPLIT ? p.causal_off : seq_k(w, p) - sq;
            const int i0 = w.q0 + t * w.dq;
            const int i = i0 + r;                     // query row
            const int n_t = t ? w.n1 : w.n0;

            if (n_t == 0) {
                // no key visible to any row of this sub-tile: O = 0, LSE = -inf
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
                // O_t was not used: hand it back at once so its barrier completes once per tile
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_o_free[t]));
            } else {
                float m_run = -INFINITY, l_run = 0.f;
                // Steps [0, n_full) lie wholly below the causal diagonal and inside the key range: nothing
                // to mask.  In the causal kernels the masking code sits in a loop of zero or one trips whose
                // count the compiler cannot see: a plain `if` ends up predicated into every step, and a
                // second copy of the step for the masked case is cold in the instruction cache at every
                // tile's diagonal (a masked step then took three times as long as an unmasked one).
                const int k_end = key_end(w, p);
                const int n_full = unmasked_steps<CAUSAL, SPLIT>(i0, n_t, key_begin(w), k_end, off, p.rows_per_head);
                auto step = [&](const int j, auto masked) -> bool {
                    // `masked` is a run-time bool (causal kernels) or std::true_type / std::false_type
                    constexpr bool kRuntimeFlag = std::is_same<decltype(masked), bool>::value;
                    bool need_mask;
                    if constexpr (kRuntimeFlag) need_mask = masked;
                    else need_mask = decltype(masked)::value;
                    if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 0);
                    ok = wait_bar(&bar_s[t], ns & 1, STATUS_TIMEOUT_MMA);
                    if (!ok) return false;
                    ++ns;
                    if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 1);
                    tc_fence_after();
                    uint32_t sraw[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld_x32(tS + c * 32, sraw[c]);
                    tmem_wait_ld();
                    if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 2);

                    const int j0 = key_begin(w) + j * BN;  // first key of this step
                    int lim = k_end - 1 - j0;           // columns c <= lim of this tile are visible to row i
                    if constexpr (SPLIT) {
                        const int pos = p.rows_per_head > 0 ? i % p.rows_per_head : i;  // query position of row i
                        if (CAUSAL) lim = min(lim, pos + off - j0);
                    } else {
                        if (CAUSAL) lim = min(lim, i + off - j0);
                    }

                    // ---- row maximum of the raw scores.  A masked score is simply replaced by -inf: it then
                    // drops out of the maximum and its probability exp2(-inf) is exactly 0.
                    const int mask_trips = kRuntimeFlag ? opaque(need_mask ? 1 : 0) : int(need_mask);
#pragma unroll 1
                    for (int trip = 0; trip < mask_trips; ++trip) {
#pragma unroll
                        for (int c = 0; c < 128; ++c)
                            sraw[c >> 5][c & 31] = (c <= lim) ? sraw[c >> 5][c & 31] : 0xff800000u;
                    }
                    // Row maximum of the (masked) raw scores, as scale*log2(e)*s; -inf if nothing is visible.
                    auto tile_max = [&]() -> float {
                        float e0 = -INFINITY, e1 = -INFINITY, e2 = -INFINITY, e3 = -INFINITY;
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            e0 = max3(e0, __uint_as_float(sraw[0][c]), __uint_as_float(sraw[0][c + 1]));
                            e1 = max3(e1, __uint_as_float(sraw[1][c]), __uint_as_float(sraw[1][c + 1]));
                            e2 = max3(e2, __uint_as_float(sraw[2][c]), __uint_as_float(sraw[2][c + 1]));
                            e3 = max3(e3, __uint_as_float(sraw[3][c]), __uint_as_float(sraw[3][c + 1]));
                        }
                        const float ext = fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
                        return (ext == -INFINITY) ? -INFINITY : ext * sl2;
                    };
                    // p = exp2(scale*log2e*s - m) for the whole row: P -> bf16 pairs into TMEM over the
                    // first 64 columns of S_t; returns the row sum of the fp32 probabilities.
                    auto exp_pass = [&](float m_ref) -> float {
                        const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
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
                                if (e & 2) acc1 = __fadd2_rn(acc1, pr);  // fp32 probabilities, before rounding to bf16
                                else       acc0 = __fadd2_rn(acc0, pr);
                                pk[e >> 1] = pack_bf16x2(pr.x, pr.y);
                            }
                            tmem_st_x16(tS + cc * 16, pk);
                        }
                        return (acc0.x + acc0.y) + (acc1.x + acc1.y);
                    };
                    // O <- alpha * O.  S_t(j) ready implies P_t V_{j-1} has finished (in-order tensor pipe).
                    auto rescale_o_wide = [&](float alpha) {
                        uint32_t oc[D / 32][32];
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) tmem_ld_x32(tO + c * 32, oc[c]);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) oc[c][e] = __float_as_uint(__uint_as_float(oc[c][e]) * alpha);
                            tmem_st_x32(tO + c * 32, oc[c]);
                        }
                    };

                    // ---- running maximum, moved lazily: probabilities are taken relative to m_run, which
                    // only moves when the row maximum has grown by more than the threshold
                    float alpha = 1.f, row_sum = 0.f;
                    // exact: take the maximum first, then exponentiate against it.  (The causal
                    // instantiations always do: with their masking code the second copy of the
                    // exponentiation loop costs registers and measured slower.)
                    bool exact = CAUSAL || (j == 0);
                    bool maximum_settled = false;
                    if (!exact) {
                        // Optimistic: start exponentiating against the current m_run at once and find the
                        // tile maximum alongside; only if it exceeds m_run by more than the threshold
                        // (rare after a row's first tiles) is the row redone, and O rescaled, below.
                        const float m_tile = tile_max();
                        row_sum = exp_pass(m_run);
                        const bool moved = m_tile - m_run > rescale_margin(l_run);  // also true for m_run = -inf < m_tile
                        if (__any_sync(0xffffffffu, moved)) {
                            if (moved) {
                                alpha = ex2_approx(m_run - m_tile);  // m_tile is finite here
                                m_run = m_tile;
                            }
                            exact = true;
                            maximum_settled = true;
                        }
                    }
                    if (exact) {
                        if (!maximum_settled) {
                            const float m_tile = tile_max();
                            if (j == 0) {
                                m_run = m_tile;
                            } else if (m_tile - m_run > rescale_margin(l_run)) {
                                alpha = ex2_approx(m_run - m_tile);
                                m_run = m_tile;
                            }
                        }
                        if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 3);
                        row_sum = exp_pass(m_run);
                        // O <- alpha * O after the exponentiation: the score registers are free by then, so the
                        // whole accumulator row is in flight at once (P_t V_j is not issued before this thread's
                        // arrival below).
                        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) rescale_o_wide(alpha);
                    }
                    l_run = l_run * alpha + row_sum;
                    if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 4);

                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_p[t]));
                    if (traced(n) && tracer) trace_stamp(1 + t, trace_it(n, j), 5);
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

                // ---- epilogue: O / l -> bf16 -> shared (TMA layout) -> global; LSE = ln2 * (m + log2 l)
                if (traced(n) && tracer) trace_stamp(1 + t, (n - kTraceTile) * 32 + 30, 0);
                if (ok) ok = wait_bar(&bar_o[t], n_out & 1, STATUS_TIMEOUT_MMA);
                if (traced(n) && tracer) trace_stamp(1 + t, (n - kTraceTile) * 32 + 30, 1);
                if (ok) {
                    ++n_out;
                    tc_fence_after();
                    const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
                    const float lse_row = (l_run > 0.f) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                    if (SPLIT) {
                        // partial result of this key range: normalised O in fp32 and its LSE, straight to global
                        const size_t row = (size_t(split_of(w)) * p.BH + bh) * p.Sq + i;
                        if (i < p.Sq) p.lse_partial[row] = lse_row;
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t oc[32];
                            tmem_ld_x32(tO + c * 32, oc);
                            tmem_wait_ld();
                            if (i < p.Sq) {
#pragma unroll
                                for (int e = 0; e < 32; e += 4)
                                    reinterpret_cast<float4 *>(p.o_partial + row * D + c * 32)[e >> 2] =
                                        make_float4(__uint_as_float(oc[e]) * inv_l, __uint_as_float(oc[e + 1]) * inv_l,
                                                    __uint_as_float(oc[e + 2]) * inv_l, __uint_as_float(oc[e + 3]) * inv_l);
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_o_free[t]));
                    } else {
                    if (i < sq) p.lse[lse_index(w, p, i)] = lse_row;
#pragma unroll
                    for (int x = 0; x < Cfg::kBoxes; ++x) {  // 64 columns of O at a time through the staging rows
                        uint32_t oc[2][32];
                        tmem_ld_x32(tO + x * 64, oc[0]);
                        tmem_ld_x32(tO + x * 64 + 32, oc[1]);
                        tmem_wait_ld();
                        if (x == Cfg::kBoxes - 1) {  // O_t is in registers: the next tile may overwrite it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(smem_u32(&bar_o_free[t]));
                        }
                        // Variable-length launches: a 32-row box that reaches past the sequence's last row would
                        // overwrite the next sequence's rows, so that warp stores its rows one by one instead.
                        const bool whole_box = !VARLEN || (i0 + wq * 32 + 32 <= sq);
                        // this warp's previous TMA store must have finished reading the staging rows
                        if (lane == 0 && store_pending) tma_store_wait_read();
                        __syncwarp();
#pragma unroll
                        for (int e = 0; e < 64; e += 8) {
                            const uint32_t *src = &oc[e >> 5][e & 31];
                            uint4 v4;
                            v4.x = pack_bf16x2(__uint_as_float(src[0]) * inv_l, __uint_as_float(src[1]) * inv_l);
                            v4.y = pack_bf16x2(__uint_as_float(src[2]) * inv_l, __uint_as_float(src[3]) * inv_l);
                            v4.z = pack_bf16x2(__uint_as_float(src[4]) * inv_l, __uint_as_float(src[5]) * inv_l);
                            v4.w = pack_bf16x2(__uint_as_float(src[6]) * inv_l, __uint_as_float(src[7]) * inv_l);
                            // 16-byte chunk `ch` of row `lane`, in the 128-byte-swizzled layout TMA expects
                            const int ch = e >> 3;
                            if (whole_box) {
                                const uint32_t addr = sO + lane * 128 + ((ch ^ (lane & 7)) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v4.x), "r"(v4.y),
                                             "r"(v4.z), "r"(v4.w) : "memory");
                            } else if (i < sq && x * 64 + e < p.d_true) {
                                __nv_bfloat16 *o_row = reinterpret_cast<__nv_bfloat16 *>(p.o) + w.h * p.o_stride_h +
                                                       (q_base_of(w) + i) * p.o_stride_r;
                                *reinterpret_cast<uint4 *>(o_row + x * 64 + e) = v4;
                            }
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0 && whole_box && i0 + wq * 32 < sq) {
                            tma_store_4d(&tm_o, sO, x * 64, q_base_of(w) + i0 + wq * 32, w.h, batch_coord(w));
                            tma_store_commit();
                            store_pending = true;
                        }
                    }
                    }
                }
            }
            if (traced(n) && tracer) trace_stamp(1 + t, (n - kTraceTile) * 32 + 30, 2);
            if (ok) id = next_tile(n, ok, w_tile);
            if (traced(n) && tracer) trace_stamp(1 + t, (n - kTraceTile) * 32 + 30, 3);
        }
        if (lane == 0 && store_pending) tma_store_wait_all();
    }

    // ---- common exit: every thread arrives, then TMEM is released
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, Cfg::kTmemCols);
    if (threadIdx.x == 0) span_stamp(1);
}

}  // namespace ave
