// Attention forward, bring-up kernel: one 128-row query tile per CTA, four
// warps that all do the same thing in lock step (no role specialisation),
// K/V double-buffered by TMA, both products on tcgen05 with accumulators in
// TMEM.  Steps follow the flash-attention loop of the paper's Section 2 and
// Fig. 1: load a Q block once, stream K/V blocks, S = Q K^T, online softmax
// with rescaling of O, O += P V, final normalisation.
#pragma once

#include "attn_common.cuh"

namespace ave {

template <int D>
struct SimpleCfg {
    static constexpr int kThreads = 128;
    static constexpr int kTileBytes = BM * D * 2;     // one Q, K or V tile
    static constexpr int kBoxBytes = BM * 64 * 2;      // one 64-column TMA box
    static constexpr int kBoxes = D / 64;
    static constexpr int kStages = 2;
    static constexpr int kSmemBytes = kTileBytes * (1 + 2 * kStages) + 1024;  // + alignment slack
    static constexpr uint32_t kTmemCols = 256;
    static constexpr uint32_t kColS = 0;    // S: 128 fp32 columns; P (bf16 pairs) reuses the first 64
    static constexpr uint32_t kColO = 128;  // O: D fp32 columns
};

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(128, 1)
attn_fwd_simple_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    using Cfg = SimpleCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[6];  // q, kv_full[2], s_done, o_done, drain
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;

    // ---- which tile (paper Fig. 1: grid = (q-block, head); here flattened, long causal blocks first)
    const int bh = blockIdx.x / p.n_qblk;
    const int qb = p.n_qblk - 1 - (blockIdx.x % p.n_qblk);
    const int b = bh / p.H;
    const int h = bh - b * p.H;
    const int g = h / (p.H / p.Hkv);           // key/value head of this query head
    const int bg = b * p.Hkv + g;
    const int i0 = qb * BM;
    const int off = p.Sk - p.Sq;                // causal: key j visible iff j <= i + off
    const int i = i0 + tid;                     // this thread's query row

    int n_kv = (p.Sk + BN - 1) / BN;
    if (CAUSAL) {
        const int i_last = min(i0 + BM, p.Sq) - 1;
        const int last_vis = i_last + off;
        n_kv = last_vis < 0 ? 0 : min(n_kv, last_vis / BN + 1);
    }
    __nv_bfloat16 *o_row = reinterpret_cast<__nv_bfloat16 *>(p.o) + (size_t(bh) * p.Sq + i) * D;
    if (n_kv == 0) {  // no row of this tile sees any key
        if (i < p.Sq) {
            const uint4 z = make_uint4(0, 0, 0, 0);
            for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4 *>(o_row)[c] = z;
            p.lse[size_t(bh) * p.Sq + i] = -INFINITY;
        }
        return;
    }

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK0 = sQ + Cfg::kTileBytes;
    const uint32_t sV0 = sK0 + Cfg::kStages * Cfg::kTileBytes;
    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_kv0 = smem_u32(&bars[1]);
    const uint32_t bar_s = smem_u32(&bars[3]);
    const uint32_t bar_o = smem_u32(&bars[4]);
    const uint32_t bar_drain = smem_u32(&bars[5]);

    if (tid == 0) {
        abort_flag = 0;
        for (int k = 0; k < 6; ++k) mbar_init(smem_u32(&bars[k]), 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const uint32_t lane_sel = uint32_t(warp * 32) << 16;  // this warp's TMEM lane quadrant
    const uint32_t tS = tmem + Cfg::kColS;
    const uint32_t tO = tmem + Cfg::kColO;

    constexpr uint32_t idesc_qk = make_idesc_bf16(BM, BN, 0);
    constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, 1);
    constexpr uint64_t desc_kmajor = make_sdesc_sw128(16, 1024);
    constexpr uint64_t desc_v = make_sdesc_sw128(BN * 128, 1024);

    int loads_issued = 0, loads_waited = 0;
    bool mma_pending = false;
    auto issue_kv = [&](int j) {
        const int st = j & 1;
        const uint32_t bar = bar_kv0 + 8u * st;
        mbar_arrive_expect_tx(bar, 2 * Cfg::kTileBytes);
        for (int x = 0; x < Cfg::kBoxes; ++x) {
            tma_load_3d(sK0 + st * Cfg::kTileBytes + x * Cfg::kBoxBytes, &tm_k, bar, x * 64, j * BN, bg);
            tma_load_3d(sV0 + st * Cfg::kTileBytes + x * Cfg::kBoxBytes, &tm_v, bar, x * 64, j * BN, bg);
        }
        ++loads_issued;
    };

    if (tid == 0) {
        mbar_arrive_expect_tx(bar_q, Cfg::kTileBytes);
        for (int x = 0; x < Cfg::kBoxes; ++x) tma_load_3d(sQ + x * Cfg::kBoxBytes, &tm_q, bar_q, x * 64, i0, bh);
        issue_kv(0);
    }

    float m_run = -INFINITY;  // running row maximum of scale*log2(e)*s
    float l_run = 0.f;        // running row sum of exp2(t - m_run)
    const bool neg = p.scale_log2 < 0.f;
    bool ok = true;

    ok = mbar_wait_bounded(bar_q, 0, &abort_flag, STATUS_TIMEOUT_LOAD);
    if (__syncthreads_or(!ok)) goto teardown;

    for (int j = 0; j < n_kv; ++j) {
        const int st = j & 1;
        if (tid == 0 && j + 1 < n_kv) issue_kv(j + 1);  // stage st^1 was released by o_done of step j-1
        ok = mbar_wait_bounded(bar_kv0 + 8u * st, (j >> 1) & 1, &abort_flag, STATUS_TIMEOUT_LOAD);
        if (tid == 0 && ok) ++loads_waited;
        if (__syncthreads_or(!ok)) goto teardown;

        // ---- S = Q K^T  (reduction over D in steps of 16)
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t koff = (kk / 4) * Cfg::kBoxBytes + (kk % 4) * 32;
                umma_ss(tS, sdesc_at(desc_kmajor, sQ + koff),
                        sdesc_at(desc_kmajor, sK0 + st * Cfg::kTileBytes + koff), idesc_qk, kk > 0);
            }
            umma_commit(bar_s);
            mma_pending = true;
        }
        ok = mbar_wait_bounded(bar_s, j & 1, &abort_flag, STATUS_TIMEOUT_MMA);
        if (tid == 0 && ok) mma_pending = false;
        if (__syncthreads_or(!ok)) goto teardown;
        tc_fence_after();

        // ---- this thread's score row
        uint32_t sraw[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_x32(tS + lane_sel + c * 32, sraw[c]);
        tmem_wait_ld();

        const int j0 = j * BN;
        // columns c <= lim of this tile are visible to row i
        int lim = p.Sk - 1 - j0;
        if (CAUSAL) lim = min(lim, i + off - j0);
        const bool need_mask = (j0 + BN > p.Sk) || (CAUSAL && (j0 + BN - 1 > i0 + off));

        float ext = neg ? INFINITY : -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; ++c) {
            const float s = __uint_as_float(sraw[c >> 5][c & 31]);
            const bool vis = !need_mask || (c <= lim);
            if (neg) ext = vis ? fminf(ext, s) : ext;
            else     ext = vis ? fmaxf(ext, s) : ext;
        }
        const float m_tile = (fabsf(ext) == INFINITY) ? -INFINITY : ext * p.scale_log2;
        const float m_new = fmaxf(m_run, m_tile);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ex2_approx(m_run - m_use);
        float rowsum = 0.f;
        uint32_t pk[2][32];
#pragma unroll
        for (int c = 0; c < 128; c += 2) {
            const float s0 = __uint_as_float(sraw[c >> 5][c & 31]);
            const float s1 = __uint_as_float(sraw[c >> 5][(c & 31) + 1]);
            float p0 = ex2_approx(fmaf(s0, p.scale_log2, -m_use));
            float p1 = ex2_approx(fmaf(s1, p.scale_log2, -m_use));
            if (need_mask) {
                p0 = (c <= lim) ? p0 : 0.f;
                p1 = (c + 1 <= lim) ? p1 : 0.f;
            }
            rowsum += p0 + p1;  // fp32 probabilities, before rounding to bf16
            pk[c >> 6][(c >> 1) & 31] = pack_bf16x2(p0, p1);
        }
        l_run = l_run * alpha + rowsum;
        m_run = m_new;

        // ---- O <- alpha * O (after the first step, when some row of the warp moved its maximum)
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t oc[32];
                tmem_ld_x32(tO + lane_sel + c * 32, oc);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) oc[e] = __float_as_uint(__uint_as_float(oc[e]) * alpha);
                tmem_st_x32(tO + lane_sel + c * 32, oc);
            }
        }
        // ---- P (bf16 pairs) over the first 64 columns of S
        tmem_st_x32(tS + lane_sel, pk[0]);
        tmem_st_x32(tS + lane_sel + 32, pk[1]);
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();

        // ---- O += P V  (reduction over the 128 keys in steps of 16)
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk) {
                umma_ts(tO, tS + kk * 8, sdesc_at(desc_v, sV0 + st * Cfg::kTileBytes + kk * 16 * 128), idesc_pv,
                        (j > 0 || kk > 0));
            }
            umma_commit(bar_o);
            mma_pending = true;
        }
        ok = mbar_wait_bounded(bar_o, j & 1, &abort_flag, STATUS_TIMEOUT_MMA);
        if (tid == 0 && ok) mma_pending = false;
        if (__syncthreads_or(!ok)) goto teardown;
        tc_fence_after();
    }

    // ---- epilogue: O / l -> bf16, LSE = ln2 * (m + log2 l)
    {
        const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            uint32_t oc[32];
            tmem_ld_x32(tO + lane_sel + c * 32, oc);
            tmem_wait_ld();
            if (i < p.Sq) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(oc[e + 0]) * inv_l, __uint_as_float(oc[e + 1]) * inv_l);
                    w.y = pack_bf16x2(__uint_as_float(oc[e + 2]) * inv_l, __uint_as_float(oc[e + 3]) * inv_l);
                    w.z = pack_bf16x2(__uint_as_float(oc[e + 4]) * inv_l, __uint_as_float(oc[e + 5]) * inv_l);
                    w.w = pack_bf16x2(__uint_as_float(oc[e + 6]) * inv_l, __uint_as_float(oc[e + 7]) * inv_l);
                    reinterpret_cast<uint4 *>(o_row)[(c * 32 + e) / 8] = w;
                }
            }
        }
        if (i < p.Sq)
            p.lse[size_t(bh) * p.Sq + i] =
                (l_run > 0.f) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
    }

teardown:
    // After an abandoned wait: give this CTA's outstanding loads and MMAs a
    // bounded chance to land before shared memory and TMEM are released.
    if (tid == 0 && abort_flag != 0) {
        for (int n = loads_waited; n < loads_issued; ++n)
            for (uint32_t it = 0; it < WAIT_LIMIT && !mbar_try_wait(bar_kv0 + 8u * (n & 1), (n >> 1) & 1); ++it) {}
        if (mma_pending) {
            umma_commit(bar_drain);
            for (uint32_t it = 0; it < WAIT_LIMIT && !mbar_try_wait(bar_drain, 0); ++it) {}
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace ave
