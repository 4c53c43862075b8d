"""Partition of an attention problem over ranks (one process per GPU).

The forward pass has no exchange step: a unit of work is one (batch, KV head)
pair together with the H/Hkv query heads that read it, and units are
independent.  Each rank calls the library on its own contiguous slice of units;
nothing crosses ranks on the data path.
"""
from __future__ import annotations


def unit_range(n_units: int, world: int, rank: int):
    """Contiguous [lo, hi) of units for `rank`; sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_qkv(q, k, v, world: int, rank: int):
    """Slices of q [B,H,Sq,D], k/v [B,Hkv,Sk,D] for `rank`, as views shaped
    [units, G, Sq, D] and [units, 1, Sk, D] (units = this rank's (b, kv head)
    pairs), which the library accepts as B=units, H=G, Hkv=1."""
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    G = H // Hkv
    lo, hi = unit_range(B * Hkv, world, rank)
    qu = q.reshape(B * Hkv, G, Sq, D)[lo:hi]
    ku = k.reshape(B * Hkv, 1, Sk, D)[lo:hi]
    vu = v.reshape(B * Hkv, 1, Sk, D)[lo:hi]
    return qu, ku, vu, (lo, hi)
