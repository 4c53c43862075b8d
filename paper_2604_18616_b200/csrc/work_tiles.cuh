// Work decomposition of the attention forward: which (batch, head, query block, key range) a CTA
// index stands for, which key/value head it reads (Fig. 1: idx_h / gqa), how many key tiles each
// of its two 128-row sub-tiles visits under the causal mask, and how many of those steps need no
// masking at all.  Integer arithmetic only and no CUDA types, so the same code compiles for the
// device (the kernels) and for the host (the launch planner, and unit tests that enumerate the
// mask by brute force).
#pragma once

#include <cstddef>
#include <type_traits>

#if defined(__CUDACC__)
#define AVE_HD __host__ __device__ __forceinline__
#else
#define AVE_HD inline
#endif

namespace ave {

constexpr int BM = 128;  // query rows per MMA tile (= TMEM lanes)
constexpr int BN = 128;  // keys per step

AVE_HD int imin(int a, int b) { return a < b ? a : b; }
AVE_HD int imax(int a, int b) { return a > b ? a : b; }

struct FwdParams {
    void *o;          // bf16 [B, H, Sq, D] through the strides below
    float *lse;       // fp32 [B, H, Sq]
    long long o_stride_b, o_stride_h, o_stride_r;  // element strides of o (rows written without TMA use them)
    int d_true;       // head dimension of the tensors (<= the kernel's D; TMA zero-fills / clips the rest)
    int H, Hkv;       // query heads, key/value heads
    int Sq, Sk;       // sequence lengths
    int BH;           // B * H
    int n_qblk;       // work tiles (blocks of query rows) per unit
    int total_blocks; // grid size: n_qblk * n_units * n_splits
    int pair_heads;   // != 0: a work tile is 128 query rows of two neighbouring query heads of one key/value head
    int one_subtile;  // != 0: a work tile is 128 query rows of one head (the single-sub-tile kernel, two CTAs per SM)
    int n_units;      // BH, or BH / 2 when heads are paired
    int heads_per_group;  // units ((b, h) pairs, or pairs of heads) whose work tiles are launched together (their K/V share L2)
    float scale_log2; // scale * log2(e)
    int causal_off;   // key j is visible to query i iff j <= i + causal_off (Sk - Sq of the whole problem)
    // Split-KV launches only: the keys are cut into n_splits ranges of keys_per_split (a multiple of
    // BN); a work tile handles one range and writes a normalised fp32 partial result.
    int n_splits;
    int keys_per_split;
    int rows_per_head;   // > 0: rows are (query head in group, query position) pairs, this many positions per head
    // Variable-length launches only: sequence b owns query rows [cu_q[b], cu_q[b+1]) and key rows
    // [cu_k[b], cu_k[b+1]) of token-major tensors [rows, heads, D]; Sq and Sk above are the maxima.
    const int *cu_q, *cu_k;        // device, B + 1 entries each
    long long lse_stride_h;        // lse is [H, total query rows]
    float *o_partial;    // fp32 [n_splits, B*H, Sq, D]
    float *lse_partial;  // fp32 [n_splits, B*H, Sq]
};

// One work tile, decoded from its position in the launch order.
struct WorkTileBase {
    int bh;      // b * H + h
    int b, h;    // batch and query head
    int g;       // h / (H / Hkv): key/value head (Fig. 1: idx_h / gqa)
    int q0;      // first query row
    int dq, dh;  // sub-tile 1 relative to sub-tile 0: rows further down (BM, same head) or, in launches that
                 // pair heads, the next query head of the same key/value head (same rows)
    int n0, n1;  // key tiles the two sub-tiles visit (n1 >= n0)
};
template <bool SPLIT>
struct WorkTileT : WorkTileBase {};
template <>
struct WorkTileT<true> : WorkTileBase {
    int k_begin, k_end;  // keys [k_begin, k_end) belong to this tile (split-KV only; else the whole range)
    int split;           // index of the key range
};

// Variable-length launches (never split): the tile also carries its sequence's lengths and first rows.
struct WorkTileVar : WorkTileT<false> {
    int sq, sk;          // this sequence's query and key counts
    int q_base, k_base;  // its first row in the token-major Q/O and K/V tensors
};
template <bool SPLIT, bool VARLEN>
using TileOf = std::conditional_t<VARLEN, WorkTileVar, WorkTileT<SPLIT>>;

// Split-KV launches may pack the G query heads of a key/value head into the rows of one problem
// ("head" = KV head, row r = head_in_group * rows_per_head + query position): the rows of Q, O and LSE
// are contiguous that way, and only the causal mask needs the query position r % rows_per_head.
// Smallest and one-past-largest query position among the rows [i0, i0 + BM):
AVE_HD int query_pos_lo(int i0, int rows_per_head) {
    if (rows_per_head <= 0) return i0;
    const int lo = i0 % rows_per_head;
    return (lo + BM > rows_per_head) ? 0 : lo;
}
AVE_HD int query_pos_hi(int i0, int rows_per_head) {
    if (rows_per_head <= 0) return i0 + BM;
    const int lo = i0 % rows_per_head;
    return (lo + BM >= rows_per_head) ? rows_per_head : lo + BM;
}

// Number of key tiles a 128-row sub-tile must visit inside [k_begin, k_end); pos_hi is one past the
// largest query position among its rows.
template <bool CAUSAL>
AVE_HD int kv_tiles_for(int pos_hi, int causal_off, int k_begin, int k_end) {
    int hi = k_end;
    if (CAUSAL) hi = imin(hi, pos_hi + causal_off);  // one past the last key any row of the sub-tile may see
    return hi > k_begin ? (hi - k_begin + BN - 1) / BN : 0;
}

// The same count when the tile covers all keys [0, Sk): key j is visible to row i iff
// j <= i + (Sk - Sq).
template <bool CAUSAL>
AVE_HD int kv_tiles_whole(int i0, int Sq, int Sk) {
    int n = (Sk + BN - 1) / BN;
    if (CAUSAL) {
        const int last_vis = i0 + BM - 1 + (Sk - Sq);  // last key the last row of the sub-tile may see
        n = last_vis < 0 ? 0 : imin(n, last_vis / BN + 1);
    }
    return n;
}

// Of the n_t key steps of a sub-tile whose rows start at i0, the first `unmasked_steps` lie wholly
// inside the key range [k_begin, k_end) and wholly below the causal diagonal of every one of its
// rows: no (row, key) pair of those steps is hidden.  `off` is the causal offset (key j visible to
// position i iff j <= i + off).
template <bool CAUSAL, bool SPLIT>
AVE_HD int unmasked_steps(int i0, int n_t, int k_begin, int k_end, int off, int rows_per_head) {
    int n_full = (k_end - k_begin) / BN;
    if (CAUSAL) {
        const int pos_lo = SPLIT ? query_pos_lo(i0, rows_per_head) : i0;
        const int num = pos_lo + off - k_begin + 1;  // keys from k_begin on that every row of the sub-tile sees
        n_full = imin(n_full, num > 0 ? num / BN : 0);
    }
    return imax(0, imin(n_full, n_t));
}

// Launch order: units ((batch, head) pairs, or pairs of heads) in groups of p.heads_per_group
// (whose K/V fit in L2 together); inside a group all units' blocks of one query position,
// longest (causal: last) position first.  Split-KV: the key ranges of one
// (b, h, block) are adjacent in the order.
template <bool CAUSAL, bool SPLIT, bool VARLEN = false>
AVE_HD TileOf<SPLIT, VARLEN> decode_tile(int id, const FwdParams &p) {
    static_assert(!(SPLIT && VARLEN), "variable-length launches are not split");
    TileOf<SPLIT, VARLEN> w;
    int k_begin = 0, k_end = p.Sk;
    if constexpr (SPLIT) {
        w.split = id % p.n_splits;
        id /= p.n_splits;
        w.k_begin = k_begin = imin(p.Sk, w.split * p.keys_per_split);
        w.k_end = k_end = imin(p.Sk, w.k_begin + p.keys_per_split);
    }
    // A unit is a (batch, head) pair or, when heads are paired, two neighbouring query heads of one
    // key/value head: the two sub-tiles then take the same 128 query rows of the two heads, so that in a
    // causal launch both visit the same key tiles and reach the diagonal, and the next tile, together.
    const bool paired = !SPLIT && p.pair_heads != 0;
    const bool single = p.one_subtile != 0;  // 128-row tiles with one sub-tile: dq = dh = 0 and n1 = n0
    const int per_group = p.heads_per_group * p.n_qblk;
    const int grp = id / per_group;
    const int rem = id - grp * per_group;
    const int u0 = grp * p.heads_per_group;
    const int hg = imin(p.heads_per_group, p.n_units - u0);
    const int rank = rem / hg;
    const int unit = u0 + (rem - rank * hg);
    w.bh = paired ? 2 * unit : unit;
    w.dq = (paired || single) ? 0 : BM;
    w.dh = paired ? 1 : 0;
    const int qb = CAUSAL ? (p.n_qblk - 1 - rank) : rank;
    w.b = w.bh / p.H;
    w.h = w.bh - w.b * p.H;
    w.g = w.h / (p.H / p.Hkv);
    w.q0 = qb * ((paired || single) ? BM : 2 * BM);
    if constexpr (SPLIT) {
        w.n0 = kv_tiles_for<CAUSAL>(query_pos_hi(w.q0, p.rows_per_head), p.causal_off, k_begin, k_end);
        w.n1 = single ? w.n0 : imax(w.n0, kv_tiles_for<CAUSAL>(query_pos_hi(w.q0 + BM, p.rows_per_head), p.causal_off, k_begin, k_end));
    } else if constexpr (VARLEN) {
        w.q_base = p.cu_q[w.b];
        w.k_base = p.cu_k[w.b];
        w.sq = p.cu_q[w.b + 1] - w.q_base;
        w.sk = p.cu_k[w.b + 1] - w.k_base;
        // sub-tiles that start beyond the sequence's last query row have no rows and visit no keys
        w.n0 = (w.q0 < w.sq && w.sk > 0) ? kv_tiles_whole<CAUSAL>(w.q0, w.sq, w.sk) : 0;
        w.n1 = (w.q0 + w.dq < w.sq && w.sk > 0) ? kv_tiles_whole<CAUSAL>(w.q0 + w.dq, w.sq, w.sk) : 0;
        w.n1 = imax(w.n0, w.n1);  // (one sub-tile: dq = 0, so n1 = n0)
    } else {
        w.n0 = kv_tiles_whole<CAUSAL>(w.q0, p.Sq, p.Sk);
        w.n1 = kv_tiles_whole<CAUSAL>(w.q0 + w.dq, p.Sq, p.Sk);
    }
    return w;
}

AVE_HD int key_begin(const WorkTileT<false> &) { return 0; }
AVE_HD int key_begin(const WorkTileT<true> &w) { return w.k_begin; }
AVE_HD int key_end(const WorkTileT<false> &, const FwdParams &p) { return p.Sk; }
AVE_HD int key_end(const WorkTileT<true> &w, const FwdParams &) { return w.k_end; }
AVE_HD int split_of(const WorkTileT<false> &) { return 0; }
AVE_HD int split_of(const WorkTileT<true> &w) { return w.split; }
AVE_HD int key_end(const WorkTileVar &w, const FwdParams &) { return w.sk; }
// Query/key counts and first rows of the tile's sequence; the tensor-map batch coordinate.
template <class Tile> AVE_HD int seq_q(const Tile &, const FwdParams &p) { return p.Sq; }
template <class Tile> AVE_HD int seq_k(const Tile &, const FwdParams &p) { return p.Sk; }
template <class Tile> AVE_HD int q_base_of(const Tile &) { return 0; }
template <class Tile> AVE_HD int k_base_of(const Tile &) { return 0; }
template <class Tile> AVE_HD int batch_coord(const Tile &w) { return w.b; }
AVE_HD int seq_q(const WorkTileVar &w, const FwdParams &) { return w.sq; }
AVE_HD int seq_k(const WorkTileVar &w, const FwdParams &) { return w.sk; }
AVE_HD int q_base_of(const WorkTileVar &w) { return w.q_base; }
AVE_HD int k_base_of(const WorkTileVar &w) { return w.k_base; }
AVE_HD int batch_coord(const WorkTileVar &) { return 0; }
// Index of row i's log-sum-exp: [B, H, Sq], or [H, total rows] for variable-length launches.
template <class Tile>
AVE_HD size_t lse_index(const Tile &w, const FwdParams &p, int i) {
    return size_t(w.bh) * p.Sq + i;
}
AVE_HD size_t lse_index(const WorkTileVar &w, const FwdParams &p, int i) {
    return size_t(w.h) * p.lse_stride_h + w.q_base + i;
}

// Host side of the decomposition: the fields of FwdParams that fix the grid and the launch order.
// `split` launches cut the keys into n_splits ranges of keys_per_split; rows_per_head > 0 marks a
// split launch whose rows pack the query heads of a key/value head (H == Hkv there).  Returns false
// when the grid would not fit in 31 bits.
inline bool plan_work_tiles(FwdParams &p, int B, int H, int Hkv, int Sq, int Sk, int D, bool causal, bool split,
                            int n_splits, int keys_per_split, int rows_per_head, bool one_subtile = false) {
    p.H = H;
    p.Hkv = Hkv;
    p.Sq = Sq;
    p.Sk = Sk;
    p.BH = B * H;
    const int G = H / Hkv;
    // Causal launches with an even number of query heads per key/value head give the two sub-tiles of a work
    // tile the same 128 query rows of two neighbouring heads instead of 256 rows of one head: both then visit
    // the same key tiles and finish together, where otherwise sub-tile 1 works through its diagonal step alone.
    p.one_subtile = one_subtile ? 1 : 0;
    p.pair_heads = (causal && !split && rows_per_head == 0 && G % 2 == 0 && !one_subtile) ? 1 : 0;
    p.n_units = p.pair_heads ? p.BH / 2 : p.BH;
    const int rows_per_tile = (p.pair_heads || one_subtile) ? BM : 2 * BM;
    p.n_qblk = (Sq + rows_per_tile - 1) / rows_per_tile;
    p.causal_off = Sk - (rows_per_head > 0 ? rows_per_head : Sq);
    p.rows_per_head = rows_per_head;
    p.n_splits = split ? n_splits : 1;
    p.keys_per_split = split ? keys_per_split : Sk;
    const long long total = (long long)p.n_qblk * p.n_units * p.n_splits;
    if (total >= (1ll << 31)) return false;
    p.total_blocks = int(total);
    // Launch units in groups whose K and V together stay within a slice of L2, whole key/value heads
    // at a time: 32 MB, which keeps the re-reads of a group's K/V in L2 (measured on D = 64, long
    // non-causal sequences: +3 % over 64 MB), unless that leaves a group with fewer than about three
    // waves of work tiles on a 148-SM part (short sequences, many heads), where 64 MB measured better.
    const long long kv_bytes_per_kv_head = 2ll * Sk * D * 2;
    auto units_for = [&](long long budget) {
        long long kv_heads = budget / kv_bytes_per_kv_head;
        if (kv_heads < 1) kv_heads = 1;
        long long upg = kv_heads * G / (p.pair_heads ? 2 : 1);
        return upg > p.n_units ? (long long)p.n_units : upg;
    };
    long long upg = units_for(32ll << 20);
    if (upg * p.n_qblk < 448) upg = units_for(64ll << 20);
    p.heads_per_group = int(upg);
    return true;
}

// Split-KV launches: keys per range = an equal share of Sk rounded up to whole key tiles.
inline int splitkv_keys_per_split(int Sk, int n_splits) {
    const long long share = ((long long)Sk + n_splits - 1) / n_splits;
    return int((share + BN - 1) / BN * BN);
}

// With grouped-query heads and few query rows, a split-KV launch turns the G query heads of a KV head into
// rows of one problem with Hkv heads of G * Sq rows each: Q, O, LSE and the partials are laid out exactly
// the same in memory, and one work tile then serves up to 256 / Sq query heads per pass over K/V.
inline bool splitkv_packs_heads(int H, int Hkv, int Sq) {
    const int G = H / Hkv;
    return G > 1 && Sq < 2 * BM && (long long)G * Sq < (1ll << 30);
}

// A default number of key ranges for a split-KV launch on a part with `sms` SMs: the largest count with
// which all work tiles are still resident at once (one CTA per SM for 256-row tiles, two for problems of at
// most 128 rows, which run the single-sub-tile kernel), so that the whole launch is one wave; measured on
// decode shapes, a second, partial wave costs more than longer key ranges do.  No range shorter than two
// key tiles.
inline int splitkv_default_splits(int B, int H, int Hkv, int Sq, int Sk, int sms, int max_splits) {
    const int G = H / Hkv;
    const bool pack = splitkv_packs_heads(H, Hkv, Sq);
    const long long rows = pack ? (long long)G * Sq : Sq;
    const bool one = rows <= BM;
    const long long rows_per_tile = one ? BM : 2 * BM;
    const long long units = (long long)B * (pack ? Hkv : H) * ((rows + rows_per_tile - 1) / rows_per_tile);
    const long long resident = one ? 2ll * sms : sms;
    const long long key_tiles = ((long long)Sk + BN - 1) / BN;
    long long n = resident / units;
    if (n > key_tiles / 2) n = key_tiles / 2;
    if (n > max_splits) n = max_splits;
    return n < 1 ? 1 : int(n);
}

}  // namespace ave
