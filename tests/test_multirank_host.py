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
