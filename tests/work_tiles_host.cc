// Host build of the attention kernels' work decomposition, for the unit tests: the library's own
// header (paper_2604_18616_b200/csrc/work_tiles.cuh) compiled with the host compiler and exposed
// through a flat C interface.  Nothing here re-implements the decomposition.
#include "../paper_2604_18616_b200/csrc/work_tiles.cuh"

extern "C" {

struct WtPlan {
    int pair_heads, n_units, n_qblk, total_blocks, heads_per_group, causal_off, n_splits, keys_per_split,
        rows_per_head, packed;  // packed: the split launch turned the query heads of a KV head into rows
    int H, Hkv, Sq;             // the problem as launched (after packing)
};

struct WtTile {
    int b, h, g, q0, dq, dh, n0, n1, k_begin, k_end, split;
    int sq, sk, q_base, k_base;   // the tile's sequence (variable-length launches; else Sq, Sk, 0, 0)
    int n_full0, n_full1;         // unmasked steps of the two sub-tiles, as the softmax warps compute them
};

}  // extern "C"

namespace {

bool g_one_subtile = false;  // plan launches for the single-sub-tile kernel (128-row tiles)

struct Launch {
    ave::FwdParams p{};
    bool causal, split, varlen;
    int packed;
};

// The same sequence of decisions the library takes in run_splitkv / launch_attention.
bool make_launch(Launch &L, int B, int H, int Hkv, int Sq, int Sk, int D, int causal, int n_splits, int varlen,
                 const int *cu_q, const int *cu_k) {
    L.causal = causal != 0;
    L.split = n_splits > 0;
    L.varlen = varlen != 0;
    L.packed = 0;
    int rows_per_head = 0, kps = 0;
    if (L.split) {
        kps = ave::splitkv_keys_per_split(Sk, n_splits);
        if (ave::splitkv_packs_heads(H, Hkv, Sq)) {
            L.packed = 1;
            rows_per_head = Sq;
            Sq = (H / Hkv) * Sq;
            H = Hkv;
        }
    }
    L.p.cu_q = cu_q;
    L.p.cu_k = cu_k;
    return ave::plan_work_tiles(L.p, B, H, Hkv, Sq, Sk, D, L.causal, L.split, n_splits, kps, rows_per_head, g_one_subtile);
}

template <bool CAUSAL, bool SPLIT, bool VARLEN>
void decode_all(const Launch &L, WtTile *out) {
    const ave::FwdParams &p = L.p;
    for (int id = 0; id < p.total_blocks; ++id) {
        const auto w = ave::decode_tile<CAUSAL, SPLIT, VARLEN>(id, p);
        WtTile &t = out[id];
        t.b = w.b; t.h = w.h; t.g = w.g; t.q0 = w.q0; t.dq = w.dq; t.dh = w.dh; t.n0 = w.n0; t.n1 = w.n1;
        t.k_begin = ave::key_begin(w);
        t.k_end = ave::key_end(w, p);
        t.split = ave::split_of(w);
        t.sq = ave::seq_q(w, p);
        t.sk = ave::seq_k(w, p);
        t.q_base = ave::q_base_of(w);
        t.k_base = ave::k_base_of(w);
        const int off = SPLIT ? p.causal_off : t.sk - t.sq;
        t.n_full0 = ave::unmasked_steps<CAUSAL, SPLIT>(w.q0, w.n0, t.k_begin, t.k_end, off, p.rows_per_head);
        t.n_full1 = ave::unmasked_steps<CAUSAL, SPLIT>(w.q0 + w.dq, w.n1, t.k_begin, t.k_end, off, p.rows_per_head);
    }
}

}  // namespace

extern "C" {

// Plan for the single-sub-tile kernel (nonzero) or the two-sub-tile kernel (zero, the default).
void wt_set_one_subtile(int on) { g_one_subtile = on != 0; }

// n_splits = 0: the ordinary forward; > 0: a split-KV launch.  varlen != 0: cu_q / cu_k are host arrays of
// B + 1 offsets and Sq / Sk the longest sequences.  Returns 0, or 1 if the grid does not fit.
int wt_plan(int B, int H, int Hkv, int Sq, int Sk, int D, int causal, int n_splits, int varlen, const int *cu_q,
            const int *cu_k, WtPlan *out) {
    Launch L;
    if (!make_launch(L, B, H, Hkv, Sq, Sk, D, causal, n_splits, varlen, cu_q, cu_k)) return 1;
    const ave::FwdParams &p = L.p;
    *out = WtPlan{p.pair_heads, p.n_units, p.n_qblk, p.total_blocks, p.heads_per_group, p.causal_off, p.n_splits,
                  p.keys_per_split, p.rows_per_head, L.packed, p.H, p.Hkv, p.Sq};
    return 0;
}

// Decodes every CTA index of the launch into out[0 .. total_blocks).
int wt_decode_all(int B, int H, int Hkv, int Sq, int Sk, int D, int causal, int n_splits, int varlen, const int *cu_q,
                  const int *cu_k, WtTile *out) {
    Launch L;
    if (!make_launch(L, B, H, Hkv, Sq, Sk, D, causal, n_splits, varlen, cu_q, cu_k)) return 1;
    if (L.varlen) {
        if (L.causal) decode_all<true, false, true>(L, out);
        else decode_all<false, false, true>(L, out);
    } else if (L.split) {
        if (L.causal) decode_all<true, true, false>(L, out);
        else decode_all<false, true, false>(L, out);
    } else {
        if (L.causal) decode_all<true, false, false>(L, out);
        else decode_all<false, false, false>(L, out);
    }
    return 0;
}

}  // extern "C"
