"""Head sharding for more than one GPU (host logic only; no arithmetic of the method).

KV groups are independent: the attention of a query head needs only its own KV head, dK / dV of a
KV head collect only from the query heads of its group.  A rank that holds the heads of a contiguous
block of KV groups, Q / O / dO / dQ as [T, Hq_local, D] and K / V / dK / dV as [T, Hkv_local, D],
therefore runs the library unchanged on its slice, and the ranks exchange nothing.
"""
from __future__ import annotations


def kv_group_shard(n_q_heads: int, n_kv_heads: int, rank: int, world: int):
    """Head ranges of `rank` out of `world`: ((q_begin, q_end), (kv_begin, kv_end)).

    KV groups are dealt out in contiguous, balanced blocks (the first n_kv_heads % world ranks get
    one more); a rank past the number of groups gets empty ranges."""
    if n_q_heads % n_kv_heads:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    g = n_q_heads // n_kv_heads
    base, extra = divmod(n_kv_heads, world)
    kv_b = rank * base + min(rank, extra)
    kv_e = kv_b + base + (1 if rank < extra else 0)
    return (kv_b * g, kv_e * g), (kv_b, kv_e)
