"""Host unit tests of the kernels' work decomposition (paper Fig. 1: grid = (query block, head),
key/value head = idx_h / gqa; causal tiles above the diagonal are skipped).

The library's own header is compiled for the host (tests/work_tiles_host.cc) and every CTA index of
a launch is decoded; the result is checked against a brute-force enumeration of the mask:

* every (batch, head, query row, key range) is handled by exactly one sub-tile;
* the key/value head of a tile is h // (H // Hkv);
* a sub-tile visits enough key tiles to reach every key one of its rows may see, and no more than
  a 128-row block at that position could need;
* no (row, key) pair of a step classed "unmasked" is hidden, and every such step lies wholly inside
  the tile's key range;

for plain, head-paired, split-KV, head-packed split-KV and variable-length launches.
"""
import ctypes
import os
import subprocess

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "work_tiles_host.cc")
HDR = os.path.join(os.path.dirname(HERE), "paper_2604_18616_b200", "csrc", "work_tiles.cuh")
BM = BN = 128


class WtPlan(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "pair_heads", "n_units", "n_qblk", "total_blocks", "heads_per_group", "causal_off", "n_splits",
        "keys_per_split", "rows_per_head", "packed", "H", "Hkv", "Sq")]


class WtTile(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "b", "h", "g", "q0", "dq", "dh", "n0", "n1", "k_begin", "k_end", "split", "sq", "sk", "q_base", "k_base",
        "n_full0", "n_full1")]


@pytest.fixture(scope="module")
def wt(tmp_path_factory):
    out = os.path.join(str(tmp_path_factory.mktemp("wt")), "libwork_tiles_host.so")
    subprocess.run(["g++", "-std=c++17", "-O1", "-shared", "-fPIC", "-o", out, SRC], check=True)
    L = ctypes.CDLL(out)
    ip = ctypes.POINTER(ctypes.c_int)
    L.wt_plan.argtypes = [ctypes.c_int] * 9 + [ip, ip, ctypes.POINTER(WtPlan)]
    L.wt_decode_all.argtypes = [ctypes.c_int] * 9 + [ip, ip, ctypes.POINTER(WtTile)]
    return L


def decode(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits=0, cu_q=None, cu_k=None):
    varlen = cu_q is not None
    cq = (ctypes.c_int * (B + 1))(*cu_q) if varlen else None
    ck = (ctypes.c_int * (B + 1))(*cu_k) if varlen else None
    plan = WtPlan()
    assert wt.wt_plan(B, H, Hkv, Sq, Sk, D, int(causal), n_splits, int(varlen), cq, ck, ctypes.byref(plan)) == 0
    tiles = (WtTile * plan.total_blocks)()
    assert wt.wt_decode_all(B, H, Hkv, Sq, Sk, D, int(causal), n_splits, int(varlen), cq, ck, tiles) == 0
    return plan, list(tiles)


def visible(sq, sk, causal):
    """Brute-force mask of one sequence: vis[i, j] = key j is visible to query position i."""
    i = np.arange(sq)[:, None]
    j = np.arange(sk)[None, :]
    return (j <= i + (sk - sq)) if causal else np.ones((sq, sk), dtype=bool)


def check_launch(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits=0, cu_q=None, cu_k=None, one=False):
    wt.wt_set_one_subtile(int(one))
    try:
        plan, tiles = decode(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits, cu_q, cu_k)
    finally:
        wt.wt_set_one_subtile(0)
    varlen = cu_q is not None
    G = H // Hkv
    ns = max(1, n_splits)
    assert plan.total_blocks == plan.n_qblk * plan.n_units * ns == len(tiles)
    if n_splits:
        assert plan.keys_per_split % BN == 0 and plan.keys_per_split * n_splits >= Sk
        assert plan.packed == int(G > 1 and Sq < 2 * BM)
    elif one:
        assert plan.pair_heads == 0 and plan.n_qblk == -(-Sq // BM)
    else:
        assert plan.pair_heads == int(bool(causal) and G % 2 == 0)
    seq = [(cu_q[b + 1] - cu_q[b], cu_k[b + 1] - cu_k[b]) for b in range(B)] if varlen else [(Sq, Sk)] * B
    masks = {s: visible(s[0], s[1], causal) for s in set(seq)}
    cover = np.zeros((B, H, Sq, ns), dtype=np.int32)   # times each (b, head, query position, key range) is handled

    for w in tiles:
        sq, sk = seq[w.b]
        assert (w.sq, w.sk) == ((G * sq if plan.packed else sq), sk)
        if varlen:
            assert (w.q_base, w.k_base) == (cu_q[w.b], cu_k[w.b])
        assert 0 <= w.k_begin <= w.k_end <= sk and (w.k_begin % BN == 0 or w.k_begin == sk)  # trailing ranges may be empty
        if not n_splits:
            assert (w.k_begin, w.k_end, w.split) == (0, sk, 0)
        assert w.n0 <= w.n1
        vis = masks[(sq, sk)]
        needed0 = None
        if one:  # 128-row tiles: the kernel has a single sub-tile and reads n0 only
            assert (w.dq, w.dh) == (0, 0) and w.n1 == w.n0
        for t in ((0,) if one else (0, 1)):
            head = w.h + t * w.dh
            i0 = w.q0 + t * w.dq
            n_t, n_full = (w.n1, w.n_full1) if t else (w.n0, w.n_full0)
            assert 0 <= n_full <= n_t
            rows = np.arange(i0, i0 + BM)
            if plan.packed:       # rows are (query head within the group, query position) pairs of KV head `head`
                rows = rows[rows < G * Sq]
                heads = head * G + rows // Sq
                pos = rows % Sq
                assert np.all(heads // G == head)
            else:
                rows = rows[rows < sq]
                heads = np.full(rows.shape, head)
                pos = rows
                if len(rows):
                    assert w.g == head // G, "key/value head of the tile"
            if len(rows):
                assert head < plan.H
                np.add.at(cover, (w.b, heads, pos, w.split), 1)
            # the keys of this tile's range that any of the sub-tile's rows may see
            sub = vis[pos][:, w.k_begin:w.k_end] if len(rows) else np.zeros((0, w.k_end - w.k_begin), dtype=bool)
            seen = np.flatnonzero(sub.any(axis=0))
            needed = 0 if seen.size == 0 else seen[-1] // BN + 1
            # an upper bound: what 128 rows at these positions could need if all of them existed
            phantom = np.arange(i0, i0 + BM)
            ppos = (phantom % Sq) if plan.packed else phantom
            if causal:
                hi = min(w.k_end, int(ppos.max()) + (sk - (Sq if plan.packed else sq)) + 1)
            else:
                hi = w.k_end
            needed_hi = max(0, -(-(hi - w.k_begin) // BN))
            if t == 0:
                needed0 = needed
                assert needed <= n_t <= max(needed, needed_hi), (t, n_t, needed, needed_hi)
            else:
                assert max(needed, w.n0) <= n_t <= max(needed, needed_hi, w.n0), (t, n_t, needed, needed_hi)
            # unmasked steps: wholly inside the key range, no hidden pair
            for j in range(n_full):
                a = w.k_begin + j * BN
                assert a + BN <= w.k_end, "an unmasked step reaches past the key range"
                assert vis[pos][:, a:a + BN].all(), "an unmasked step hides a (row, key) pair"
            # and the classification is not needlessly pessimistic: the first masked step really needs its mask
            # (or the sub-tile has rows that do not exist, whose positions the kernel bounds conservatively)
            if n_full < n_t and len(rows) == BM and not plan.packed:
                a = w.k_begin + n_full * BN
                blk = vis[pos][:, a:min(a + BN, w.k_end)]
                assert blk.shape[1] < BN or not blk.all()

    for b in range(B):
        sq, _ = seq[b]
        assert np.all(cover[b, :, :sq, :] == 1), "a (head, row, key range) is handled %s times" % (
            "0" if (cover[b, :, :sq, :] == 0).any() else "several")
        assert np.all(cover[b, :, sq:, :] == 0)
    return plan, tiles


def _cases(n, seed, kind):
    rng = np.random.default_rng(seed)
    edge = [1, 2, 63, 127, 128, 129, 255, 256, 257, 383, 384, 385, 511, 512, 513]
    out = []
    for _ in range(n):
        hkv = int(rng.choice([1, 2, 3]))
        g = int(rng.choice([1, 2, 3, 4, 8]))
        B = int(rng.integers(1, 4))
        sq = int(rng.choice(edge)) if rng.random() < 0.6 else int(rng.integers(1, 800))
        sk = int(rng.choice(edge)) if rng.random() < 0.6 else int(rng.integers(1, 1000))
        causal = bool(rng.random() < 0.65)
        D = int(rng.choice([64, 128]))
        if kind == "split":
            sq = int(rng.choice([1, 2, 5, 33, 64, 127, 128, 200, 255, 256, 300]))
            sk = int(rng.integers(1, 3000))
            out.append((B, hkv * g, hkv, sq, sk, D, causal, int(rng.choice([1, 2, 3, 5, 8, 16, 64]))))
        else:
            out.append((B, hkv * g, hkv, sq, sk, D, causal))
    return out


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", _cases(140, 11, "plain"))
def test_plain_and_head_paired_launches(wt, B, H, Hkv, Sq, Sk, D, causal):
    check_launch(wt, B, H, Hkv, Sq, Sk, D, causal)


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,n_splits", _cases(90, 12, "split"))
def test_split_kv_launches_with_and_without_packed_heads(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits):
    check_launch(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits=n_splits)


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", _cases(60, 21, "plain"))
def test_single_sub_tile_launches(wt, B, H, Hkv, Sq, Sk, D, causal):
    check_launch(wt, B, H, Hkv, Sq, Sk, D, causal, one=True)


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal,n_splits", _cases(40, 22, "split"))
def test_single_sub_tile_split_kv_launches(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits):
    check_launch(wt, B, H, Hkv, Sq, Sk, D, causal, n_splits=n_splits, one=True)


def _varlen_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        B = int(rng.integers(1, 6))
        hkv = int(rng.choice([1, 2]))
        g = int(rng.choice([1, 2, 4]))
        lq = [int(rng.choice([0, 1, 100, 128, 129, 256, 300, 513])) if rng.random() < 0.5 else int(rng.integers(0, 600))
              for _ in range(B)]
        same = rng.random() < 0.5
        lk = lq if same else [int(rng.integers(0, 700)) for _ in range(B)]
        if max(lq) == 0:
            lq[0] = 7
        if max(lk) == 0:
            lk = list(lk)
            lk[0] = 9
        out.append((B, hkv * g, hkv, lq, list(lk), bool(rng.random() < 0.6)))
    return out


@pytest.mark.parametrize("B,H,Hkv,lq,lk,causal", _varlen_cases(60, 13))
def test_variable_length_launches(wt, B, H, Hkv, lq, lk, causal):
    cu_q = np.concatenate([[0], np.cumsum(lq)]).tolist()
    cu_k = np.concatenate([[0], np.cumsum(lk)]).tolist()
    check_launch(wt, B, H, Hkv, max(lq), max(lk), 128, causal, cu_q=cu_q, cu_k=cu_k)
    check_launch(wt, B, H, Hkv, max(lq), max(lk), 128, causal, cu_q=cu_q, cu_k=cu_k, one=True)


def test_the_five_configurations_and_the_papers_shape(wt):
    """Launch geometry of the named workloads: grid sizes and the longest-first order of causal tiles."""
    # c2: causal MHA, no heads to pair -> 256-row tiles; 4*32 units x 8 blocks
    plan, tiles = decode(wt, 4, 32, 32, 2048, 2048, 128, True)
    assert (plan.pair_heads, plan.n_qblk, plan.total_blocks) == (0, 8, 1024)
    assert tiles[0].q0 == 2048 - 256 and tiles[0].n1 == 16          # the longest tiles of a group come first
    # c3: causal GQA, 8 query heads per KV head -> two heads per tile, 128 rows
    plan, tiles = decode(wt, 2, 64, 8, 4096, 4096, 128, True)
    assert (plan.pair_heads, plan.n_units, plan.n_qblk) == (1, 64, 32)
    assert all(t.dh == 1 and t.dq == 0 and t.n0 == t.n1 for t in tiles[:200])
    assert all(t.g == t.h // 8 == (t.h + 1) // 8 for t in tiles)
    # the paper's shape: batch 16, 8 query heads on 1 KV head
    plan, tiles = decode(wt, 16, 8, 1, 1024, 1024, 128, True)
    assert plan.pair_heads == 1 and plan.total_blocks == 16 * 4 * 8
    # c5: non-causal, D = 64: every tile visits all 64 key tiles, none masked
    plan, tiles = decode(wt, 8, 16, 16, 8192, 8192, 64, False)
    assert all(t.n0 == t.n1 == 64 == t.n_full0 == t.n_full1 for t in tiles[::97])
