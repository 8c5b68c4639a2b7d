"""GPU: head shards reproduce the whole.  What every rank of a head-sharded run would compute (its
block of KV groups, as contiguous [T, H_local, D] tensors) is run shard by shard on one GPU and
compared with the unsharded call: O and LSE bit for bit (the kernels take heads independently),
dQ, dK and dV within a bf16 unit (their fp32 sums are formed by reductions in no fixed order)."""
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from paper_2602_01469_b200.sharding import kv_group_shard
from tests.gpu_common import DeviceCase

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3])
def test_head_shards_reproduce_the_whole(world):
    ctx = binding.Context(0)
    w = inputs.Workload("shards", (600,), 4, 12, 6, 64, n_segments=2, seed=21)
    case = DeviceCase(w)
    binding.peagle_attn_partitioned(ctx, case.prob, case.bparts, case.dQ_, case.dK_, case.dV_,
                                    case.ddO, case.O, case.LSE, case.dQ, case.dK, case.dV)
    assert binding.peagle_poll_status(ctx) == 0
    for rank in range(world):
        (qb, qe), (kb, ke) = kv_group_shard(w.n_q_heads, w.n_kv_heads, rank, world)
        if qe == qb:
            continue
        Q, dO = case.dQ_[:, qb:qe].contiguous(), case.ddO[:, qb:qe].contiguous()
        K, V = case.dK_[:, kb:ke].contiguous(), case.dV_[:, kb:ke].contiguous()
        O, dQ = torch.empty_like(Q), torch.empty_like(Q)
        dK, dV = torch.empty_like(K), torch.empty_like(V)
        LSE = torch.empty(qe - qb, case.T, dtype=torch.float32, device="cuda")
        prob = binding.Problem(case.cu, case.d_anchor, case.d_depth, w.K, qe - qb, ke - kb,
                               w.head_dim, w.scale)
        binding.peagle_attn_partitioned(ctx, prob, case.bparts, Q, K, V, dO, O, LSE, dQ, dK, dV)
        assert binding.peagle_poll_status(ctx) == 0
        assert torch.equal(O, case.O[:, qb:qe])
        assert torch.equal(LSE, case.LSE[qb:qe])
        for got, want in ((dQ, case.dQ[:, qb:qe]), (dK, case.dK[:, kb:ke]), (dV, case.dV[:, kb:ke])):
            err = (got.float() - want.float()).abs()
            assert bool((err <= want.float().abs() * 2.0 ** -7 + 1e-6).all())
