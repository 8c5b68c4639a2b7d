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


def partition_cost(part) -> int:
    """Work estimate of a query partition {q: (b, e), k: [(b, e), ...]}: query rows times visible
    keys.  Only the ordering of the costs matters (longest first when dealing out)."""
    q_len = part["q"][1] - part["q"][0]
    return q_len * sum(e - b for b, e in part["k"])


def deal_partitions(parts, world: int):
    """Partition sharding: which rank runs which query partitions.

    Query partitions of a sequence are independent given K and V; only dK / dV of the keys that
    several partitions see (the depth-0 tokens of earlier segments) are sums over partitions, so a
    rank that runs a subset of the partitions against the full K / V produces partial fp32 dK / dV
    sums, and one sum over the ranks completes them.  The partitions are dealt out longest first,
    each to the rank with the least work so far (ties to the lowest rank), so that every rank
    derives the same assignment from the same list.  Returns ``world`` lists of indices into
    ``parts``, each in ascending order."""
    if world < 1:
        raise ValueError("world must be positive")
    load = [0] * world
    mine = [[] for _ in range(world)]
    order = sorted(range(len(parts)), key=lambda i: (-partition_cost(parts[i]), i))
    for i in order:
        r = min(range(world), key=lambda j: (load[j], j))
        mine[r].append(i)
        load[r] += partition_cost(parts[i])
    return [sorted(m) for m in mine]


def sum_over_ranks(tensors, world: int):
    """Completes the partial dK / dV sums: one all-reduce (sum) of each tensor over the process
    group (the default group; NCCL on GPUs, gloo on CPU).  A no-op on one rank."""
    if world <= 1:
        return
    import torch.distributed as dist

    for t in tensors:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
