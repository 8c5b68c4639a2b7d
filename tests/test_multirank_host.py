"""CPU, two gloo ranks: the multi-rank bookkeeping of the benchmark (replicas only: no data-path
collective; the timed figure is the slowest rank's, the value is the replicas' sum)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
        out[rank] = (ms, bench.replicas_value(world, 2.0e12, ms))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_value():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        ms, value = out[0]
        assert ms == 15.0                                   # rank 1 is the slower one
        assert value == pytest.approx(2 * 2.0 / 15.0e-3)    # two replicas' TFLOP over that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.replicas_value(1, 4.0e12, 2.0) == pytest.approx(2000.0)


def _shard_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2602_01469_b200.sharding import kv_group_shard
        mine = torch.tensor(sum(kv_group_shard(64, 8, rank, world), ()), dtype=torch.int64)
        got = [torch.zeros(4, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(got, mine)
        out[rank] = [t.tolist() for t in got]
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_kv_groups_without_overlap():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [[0, 32, 0, 4], [32, 64, 4, 8]]


def test_kv_group_shards_partition_the_heads():
    from paper_2602_01469_b200.sharding import kv_group_shard
    for hq, hkv, world in ((64, 8, 8), (64, 8, 3), (32, 4, 8), (4, 1, 2), (6, 6, 4)):
        g = hq // hkv
        q_at = kv_at = 0
        for r in range(world):
            (qb, qe), (kb, ke) = kv_group_shard(hq, hkv, r, world)
            assert (qb, kb) == (q_at, kv_at) and qe - qb == g * (ke - kb) and ke >= kb
            q_at, kv_at = qe, ke
        assert (q_at, kv_at) == (hq, hkv)
    with pytest.raises(ValueError):
        kv_group_shard(6, 4, 0, 2)


# ---------------------------------------------------------------- partition sharding
def test_deal_partitions_covers_every_partition_once_and_balances():
    from paper_2602_01469_b200 import inputs
    from paper_2602_01469_b200.sharding import deal_partitions, partition_cost
    from oracle import partition as opart
    import numpy as np

    def oracle_assign(anchor, depth, K, bounds):
        P = inputs.position_sets(anchor, depth, K)
        A, _, _ = opart.assign_segments(P, len(bounds) - 1, bounds[-1], B=bounds)
        return np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)

    _, _, _, parts = inputs.build_case(inputs.WORKLOADS["longtail_varlen"], oracle_assign)
    assert len(parts) == 19
    for world in (1, 2, 3, 8, 32):
        mine = deal_partitions(parts, world)
        assert sorted(i for m in mine for i in m) == list(range(len(parts)))
        loads = [sum(partition_cost(parts[i]) for i in m) for m in mine]
        if world <= 8:      # longest-first greedy: no rank exceeds the mean by more than one item
            assert max(loads) <= sum(loads) / world + max(partition_cost(p) for p in parts)
    with pytest.raises(ValueError):
        deal_partitions(parts, 0)


def _partition_worker(rank, world, port, out):
    """Each rank runs the fp64 oracle on its share of the partitions; the partial dK / dV sums are
    completed by the all-reduce the GPU path uses (gloo here)."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import numpy as np
        from oracle import partition as opart
        from oracle import peagle_oracle as orc
        from paper_2602_01469_b200 import inputs
        from paper_2602_01469_b200.sharding import deal_partitions, sum_over_ranks

        def oracle_assign(anchor, depth, K, bounds):
            P = inputs.position_sets(anchor, depth, K)
            A, _, _ = opart.assign_segments(P, len(bounds) - 1, bounds[-1], B=bounds)
            return np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)

        w = inputs.Workload("shard_parts", (41,), 4, 4, 2, 8, n_segments=3, seed=23)
        cu, anchor, depth, parts = inputs.build_case(w, oracle_assign)
        T = int(cu[-1])
        Q, K, V, dO = inputs.make_tensors(T, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed, q_std=1.0)
        dK = np.zeros((T, w.n_kv_heads, w.head_dim))
        dV = np.zeros_like(dK)
        dQ = np.zeros((T, w.n_q_heads, w.head_dim))
        for i in deal_partitions(parts, world)[rank]:
            rows = np.arange(*parts[i]["q"])
            dQ[rows], _, _ = orc.attn_bwd(anchor, depth, Q, K, V, dO, 0.3, rows=rows,
                                          kranges=parts[i]["k"], dK=dK, dV=dV)
        tK, tV, tQ = torch.from_numpy(dK), torch.from_numpy(dV), torch.from_numpy(dQ)
        sum_over_ranks([tK, tV, tQ], world)      # dQ rows are disjoint over ranks: the sum gathers them
        want = orc.attn_bwd(anchor, depth, Q, K, V, dO, 0.3)
        out[rank] = tuple(float(np.abs(a.numpy() - b).max()) for a, b in zip((tQ, tK, tV), want))
    finally:
        dist.destroy_process_group()


def test_two_ranks_partition_shards_sum_to_the_unpartitioned_gradients():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_partition_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            assert max(out[rank]) < 1e-11, out[rank]
