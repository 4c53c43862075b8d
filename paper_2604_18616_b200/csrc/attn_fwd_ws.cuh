// Attention forward, warp-specialised kernel for sm_100a.
//
// One CTA owns a block of 256 query rows of one (batch, head): two 128-row
// sub-tiles that ping-pong so the tensor pipe works on one while the softmax
// of the other runs (the paper's "+Pipe": software pipelining across disjoint
// groups of warps, Section 9; steps of the loop as in Section 2 / Fig. 1).
//
//   warp 0        producer: TMA loads of Q (once) and of the K/V ring
//   warp 1        MMA issuer: S_t = Q_t K_j^T and O_t += P_t V_j on tcgen05
//   warp 2        TMEM allocation / release
//   warps 4..7    softmax of sub-tile 0 (one thread per query row)
//   warps 8..11   softmax of sub-tile 1
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [384,384+D); P_t
// (bf16 pairs) overwrites the first 64 columns of S_t once a thread holds its
// whole score row in registers.
#pragma once

#include "attn_common.cuh"

namespace ave {

template <int D>
struct WsCfg {
    static constexpr int kThreads = 384;
    static constexpr int kQRows = 2 * BM;                    // query rows per CTA
    static constexpr int kTileBytes = BM * D * 2;            // one Q sub-tile, K tile or V tile
    static constexpr int kBoxBytes = BM * 64 * 2;            // one 64-column TMA box
    static constexpr int kBoxes = D / 64;
    static constexpr int kStages = (D == 128) ? 5 : 8;       // ring slots, K and V tiles alternate
    static constexpr int kSmemBytes = kTileBytes * (2 + kStages) + 1024;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kRegsLight = 64;                    // producer / MMA warpgroup
    static constexpr int kRegsSoftmax = 216;                 // softmax warpgroups
};

// Rescale O only when the running maximum moved by more than this many
// powers of two; until then probabilities are taken relative to a stale
// maximum (at most 2^8 too large), which the final division by l undoes.
constexpr float kRescaleThreshold = 8.0f;

template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Number of key tiles a 128-row sub-tile starting at row i0 must visit.
template <bool CAUSAL>
__device__ __forceinline__ int kv_tiles_for(int i0, int Sq, int Sk) {
    int n = (Sk + BN - 1) / BN;
    if (CAUSAL) {
        const int last_vis = i0 + BM - 1 + (Sk - Sq);  // last key the last row of the sub-tile may see
        n = last_vis < 0 ? 0 : min(n, last_vis / BN + 1);
    }
    return n;
}

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(384, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                   const FwdParams p) {
    using Cfg = WsCfg<D>;
    constexpr int NS = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q[2], bar_s[2], bar_p[2], bar_o[2], bar_drain;
    __shared__ __align__(8) uint64_t bar_full[NS], bar_empty[NS];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // ---- work decomposition (Fig. 1: grid = (q-block, head)); long causal blocks first
    const int bh = blockIdx.x / p.n_qblk;
    const int qb = p.n_qblk - 1 - (blockIdx.x % p.n_qblk);
    const int b = bh / p.H;
    const int h = bh - b * p.H;
    const int bg = b * p.Hkv + h / (p.H / p.Hkv);  // key/value head: idx_h / gqa
    const int q0 = qb * Cfg::kQRows;
    const int n0 = kv_tiles_for<CAUSAL>(q0, p.Sq, p.Sk);
    const int n1 = kv_tiles_for<CAUSAL>(q0 + BM, p.Sq, p.Sk);  // n1 >= n0

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;                           // two sub-tiles
    const uint32_t sRing = smem_base + 2 * Cfg::kTileBytes;  // NS slots

    if (tid == 0) {
        // A wait that ran out earlier (in this launch or a previous one) leaves the
        // status word set until the host reads it; later CTAs then skip their work
        // instead of each running into the same limit.
        abort_flag = (*reinterpret_cast<volatile unsigned int *>(&g_device_status) != 0) ? 1 : 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar_q[t]), 1);
            mbar_init(smem_u32(&bar_s[t]), 1);
            mbar_init(smem_u32(&bar_p[t]), 4);  // one arrival per softmax warp
            mbar_init(smem_u32(&bar_o[t]), 1);
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

    if (poisoned) {
        // nothing: fall through to the common exit
    } else if (warp < 4) {
        setmaxnreg_dec<Cfg::kRegsLight>();
        if (warp == 0 && lane == 0 && n1 > 0) {
            // =============================== producer ===============================
            tma_prefetch_desc(&tm_q);
            tma_prefetch_desc(&tm_k);
            tma_prefetch_desc(&tm_v);
            for (int t = 0; t < 2; ++t) {
                const uint32_t bar = smem_u32(&bar_q[t]);
                mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                for (int x = 0; x < Cfg::kBoxes; ++x)
                    tma_load_3d(sQ + t * Cfg::kTileBytes + x * Cfg::kBoxBytes, &tm_q, bar, x * 64, q0 + t * BM, bh);
            }
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < 2 * n1 && ok; ++it) {  // it even: K_{it/2}; odd: V_{it/2}
                const int slot = it % NS, round = it / NS;
                if (round > 0)
                    ok = mbar_wait_bounded(smem_u32(&bar_empty[slot]), (round - 1) & 1, &abort_flag, STATUS_TIMEOUT_SLOT);
                if (!ok) break;
                const uint32_t bar = smem_u32(&bar_full[slot]);
                const CUtensorMap *tm = (it & 1) ? &tm_v : &tm_k;
                mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
                for (int x = 0; x < Cfg::kBoxes; ++x)
                    tma_load_3d(sRing + slot * Cfg::kTileBytes + x * Cfg::kBoxBytes, tm, bar, x * 64, (it >> 1) * BN, bg);
                issued = it + 1;
            }
            if (!ok) {
                // abandoned: give the loads still in flight a bounded chance to land
                for (int it = max(0, issued - NS); it < issued; ++it)
                    for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_try_wait(smem_u32(&bar_full[it % NS]), (it / NS) & 1); ++w) {}
            }
        } else if (warp == 1 && lane == 0 && n1 > 0) {
            // =============================== MMA issuer ===============================
            constexpr uint32_t idesc_qk = make_idesc_bf16(BM, BN, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, 1);
            constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);
            constexpr uint64_t desc_v = make_sdesc_sw128(BN * 128, 1024);
            const uint32_t tS[2] = {tmem + Cfg::kColS0, tmem + Cfg::kColS1};
            const uint32_t tO[2] = {tmem + Cfg::kColO0, tmem + Cfg::kColO1};
            bool ok = true;

            auto wait_full = [&](int idx) {
                return mbar_wait_bounded(smem_u32(&bar_full[idx % NS]), (idx / NS) & 1, &abort_flag, STATUS_TIMEOUT_LOAD);
            };
            auto slot_addr = [&](int idx) { return sRing + (idx % NS) * Cfg::kTileBytes; };
            auto issue_qk = [&](int t, uint32_t k_addr) {
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = (kk / 4) * Cfg::kBoxBytes + (kk % 4) * 32;
                    umma_ss(tS[t], sdesc_at(desc_kmajor, sQ + t * Cfg::kTileBytes + koff),
                            sdesc_at(desc_kmajor, k_addr + koff), idesc_qk, kk > 0);
                }
                umma_commit(smem_u32(&bar_s[t]));
            };
            auto issue_pv = [&](int t, uint32_t v_addr, bool first) {
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
                    umma_ts(tO[t], tS[t] + kk * 8, sdesc_at(desc_v, v_addr + kk * 16 * 128), idesc_pv,
                            (!first || kk > 0));
            };

            ok = mbar_wait_bounded(smem_u32(&bar_q[0]), 0, &abort_flag, STATUS_TIMEOUT_LOAD) &&
                 mbar_wait_bounded(smem_u32(&bar_q[1]), 0, &abort_flag, STATUS_TIMEOUT_LOAD) && wait_full(0);
            if (ok) {
                tc_fence_after();
                if (n0 > 0) issue_qk(0, slot_addr(0));
                issue_qk(1, slot_addr(0));
                umma_commit(smem_u32(&bar_empty[0]));
            }
            for (int j = 0; j < n1 && ok; ++j) {
                const int iv = 2 * j + 1, ik = 2 * j + 2;  // ring indices of V_j and K_{j+1}
                if (j < n0) {
                    ok = mbar_wait_bounded(smem_u32(&bar_p[0]), j & 1, &abort_flag, STATUS_TIMEOUT_SOFTMAX) && wait_full(iv);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(0, slot_addr(iv), j == 0);
                    if (j == n0 - 1) umma_commit(smem_u32(&bar_o[0]));
                    if (j + 1 < n0) {
                        ok = wait_full(ik);
                        if (!ok) break;
                        issue_qk(0, slot_addr(ik));
                    }
                }
                ok = mbar_wait_bounded(smem_u32(&bar_p[1]), j & 1, &abort_flag, STATUS_TIMEOUT_SOFTMAX) && wait_full(iv);
                if (!ok) break;
                tc_fence_after();
                issue_pv(1, slot_addr(iv), j == 0);
                umma_commit(smem_u32(&bar_empty[iv % NS]));
                if (j == n1 - 1) umma_commit(smem_u32(&bar_o[1]));
                if (j + 1 < n1) {
                    ok = wait_full(ik);
                    if (!ok) break;
                    issue_qk(1, slot_addr(ik));
                    umma_commit(smem_u32(&bar_empty[ik % NS]));
                }
            }
            if (!ok) {  // abandoned: let the MMAs already issued finish before TMEM is released
                umma_commit(smem_u32(&bar_drain));
                for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_try_wait(smem_u32(&bar_drain), 0); ++w) {}
            }
        }
    } else {
        // =============================== softmax warpgroups ===============================
        setmaxnreg_inc<Cfg::kRegsSoftmax>();
        const int t = (warp - 4) >> 2;                // sub-tile
        const int r = tid - 128 - t * 128;            // row within the sub-tile = TMEM lane
        const int i0 = q0 + t * BM;
        const int i = i0 + r;                         // query row
        const int n_t = t ? n1 : n0;
        const int off = p.Sk - p.Sq;
        const uint32_t lane_sel = uint32_t((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + (t ? Cfg::kColS1 : Cfg::kColS0) + lane_sel;
        const uint32_t tO = tmem + (t ? Cfg::kColO1 : Cfg::kColO0) + lane_sel;
        const uint32_t sO = sQ + t * Cfg::kTileBytes;  // O staging reuses this sub-tile's Q buffer
        const float sl2 = p.scale_log2;
        const bool neg = sl2 < 0.f;

        if (n_t == 0) {
            // no key visible to any row of this sub-tile: O = 0, LSE = -inf
            if (i < p.Sq) {
                __nv_bfloat16 *o_row = reinterpret_cast<__nv_bfloat16 *>(p.o) + (size_t(bh) * p.Sq + i) * D;
                const uint4 z = make_uint4(0, 0, 0, 0);
                for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4 *>(o_row)[c] = z;
                p.lse[size_t(bh) * p.Sq + i] = -INFINITY;
            }
        } else {
            float m_run = -INFINITY, l_run = 0.f;
            bool ok = true;
            for (int j = 0; j < n_t; ++j) {
                ok = mbar_wait_bounded(smem_u32(&bar_s[t]), j & 1, &abort_flag, STATUS_TIMEOUT_MMA);
                ok = __all_sync(0xffffffffu, ok);  // keep the warp together for the .sync.aligned TMEM ops
                if (!ok) break;
                tc_fence_after();
                uint32_t sraw[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld_x32(tS + c * 32, sraw[c]);
                tmem_wait_ld();

                const int j0 = j * BN;
                int lim = p.Sk - 1 - j0;  // columns c <= lim of this tile are visible to row i
                if (CAUSAL) lim = min(lim, i + off - j0);
                const bool need_mask = (j0 + BN > p.Sk) || (CAUSAL && (j0 + BN - 1 > i0 + off));

                // ---- row extreme of the raw scores (maximum of scale*s is at max s, or min s if scale < 0)
                float ext;
                if (!need_mask && !neg) {
                    float e0 = -INFINITY, e1 = -INFINITY, e2 = -INFINITY, e3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        e0 = fmaxf(e0, __uint_as_float(sraw[0][c]));
                        e1 = fmaxf(e1, __uint_as_float(sraw[1][c]));
                        e2 = fmaxf(e2, __uint_as_float(sraw[2][c]));
                        e3 = fmaxf(e3, __uint_as_float(sraw[3][c]));
                    }
                    ext = fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
                } else {
                    ext = neg ? INFINITY : -INFINITY;
#pragma unroll
                    for (int c = 0; c < 128; ++c) {
                        const float s = __uint_as_float(sraw[c >> 5][c & 31]);
                        const bool vis = !need_mask || (c <= lim);
                        if (neg) ext = vis ? fminf(ext, s) : ext;
                        else     ext = vis ? fmaxf(ext, s) : ext;
                    }
                }
                const float m_tile = (fabsf(ext) == INFINITY) ? -INFINITY : ext * sl2;

                // ---- running maximum, moved lazily
                float alpha = 1.f;
                if (j == 0) {
                    m_run = m_tile;
                } else if (m_tile - m_run > kRescaleThreshold) {  // also true when m_run = -inf < m_tile
                    const float m_use = m_tile;                   // finite here
                    alpha = ex2_approx(m_run - m_use);
                    m_run = m_use;
                }
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    // O <- alpha * O.  S_t(j) ready implies P_t V_{j-1} has finished (in-order tensor pipe).
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t oc[32];
                        tmem_ld_x32(tO + c * 32, oc);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) oc[e] = __float_as_uint(__uint_as_float(oc[e]) * alpha);
                        tmem_st_x32(tO + c * 32, oc);
                    }
                }
                const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;

                // ---- p = exp2(scale*log2e*s - m); row sum in fp32; P -> bf16 pairs into TMEM
                float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float p0 = ex2_approx(fmaf(__uint_as_float(sraw[cc][e]), sl2, neg_m));
                        float p1 = ex2_approx(fmaf(__uint_as_float(sraw[cc][e + 1]), sl2, neg_m));
                        if (need_mask) {
                            p0 = (cc * 32 + e <= lim) ? p0 : 0.f;
                            p1 = (cc * 32 + e + 1 <= lim) ? p1 : 0.f;
                        }
                        sum0 += p0;
                        sum1 += p1;
                        pk[e >> 1] = pack_bf16x2(p0, p1);
                    }
                    tmem_st_x16(tS + cc * 16, pk);
                }
                l_run = l_run * alpha + (sum0 + sum1);

                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_p[t]));
            }

            // ---- epilogue: O / l -> bf16 -> shared (TMA layout) -> global; LSE = ln2 * (m + log2 l)
            if (ok) ok = mbar_wait_bounded(smem_u32(&bar_o[t]), 0, &abort_flag, STATUS_TIMEOUT_MMA);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t oc[32];
                    tmem_ld_x32(tO + c * 32, oc);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(oc[e + 0]) * inv_l, __uint_as_float(oc[e + 1]) * inv_l);
                        w.y = pack_bf16x2(__uint_as_float(oc[e + 2]) * inv_l, __uint_as_float(oc[e + 3]) * inv_l);
                        w.z = pack_bf16x2(__uint_as_float(oc[e + 4]) * inv_l, __uint_as_float(oc[e + 5]) * inv_l);
                        w.w = pack_bf16x2(__uint_as_float(oc[e + 6]) * inv_l, __uint_as_float(oc[e + 7]) * inv_l);
                        // 16-byte chunk `ch` of row r, in the 128-byte-swizzled box layout TMA expects
                        const int ch = (c * 32 + e) >> 3;
                        const uint32_t addr = sO + (ch >> 3) * Cfg::kBoxBytes + r * 128 + (((ch & 7) ^ (r & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w.x), "r"(w.y),
                                     "r"(w.z), "r"(w.w) : "memory");
                    }
                }
                if (i < p.Sq)
                    p.lse[size_t(bh) * p.Sq + i] =
                        (l_run > 0.f) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                fence_proxy_async_smem();
            }
            named_barrier_sync(1 + t, 128);  // reached by every thread of the warpgroup, abandoned or not
            if (r == 0 && i0 < p.Sq && abort_flag == 0) {
                for (int x = 0; x < Cfg::kBoxes; ++x) tma_store_3d(&tm_o, sO + x * Cfg::kBoxBytes, x * 64, i0, bh);
                tma_store_commit();
                tma_store_wait_all();
            }
        }
    }

    // ---- common exit: every thread arrives, then TMEM is released
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace ave
