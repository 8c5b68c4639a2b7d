"""GPU: partition shards sum to the whole.  What every rank of a partition-sharded run would do
(its share of the query partitions against the full K / V, adding into its own fp32 dK / dV
accumulators) is run rank by rank on one GPU; the accumulators are summed as the all-reduce would,
rounded by the library, and everything is compared with the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from paper_2602_01469_b200.sharding import deal_partitions
from tests.gpu_common import TOL_RELL2_GRAD, DeviceCase, check_forward, check_rows, rel_l2
from tests.test_gpu_backward import oracle_all

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3])
def test_partition_shards_sum_to_the_oracle(world):
    ctx = binding.Context(0)
    w = inputs.Workload("part_shards", (900, 300), 4, 8, 2, 64, n_segments=3, seed=22)
    case = DeviceCase(w)
    assert len(case.parts) == 6
    mine = deal_partitions(case.parts, world)
    accs = []
    for rank in range(world):
        dK_acc = torch.zeros(case.T, w.n_kv_heads, w.head_dim, dtype=torch.float32, device="cuda")
        dV_acc = torch.zeros_like(dK_acc)
        binding.peagle_attn_partitioned_acc(ctx, case.prob, [case.bparts[i] for i in mine[rank]],
                                            case.dQ_, case.dK_, case.dV_, case.ddO, case.O, case.LSE,
                                            case.dQ, dK_acc, dV_acc)
        assert binding.peagle_poll_status(ctx) == 0
        accs.append((dK_acc, dV_acc))
    dK_sum = torch.stack([a[0] for a in accs]).sum(0)       # what the all-reduce leaves on every rank
    dV_sum = torch.stack([a[1] for a in accs]).sum(0)
    binding.peagle_cast_grads(ctx, dK_sum, dV_sum, case.dK, case.dV)
    assert binding.peagle_poll_status(ctx) == 0
    O, LSE, dQ, dK, dV = oracle_all(case)
    check_forward(case.O.float().cpu().numpy(), case.LSE.t().cpu().numpy(), O, LSE)
    for name, got, want in (("dQ", case.dQ, dQ), ("dK", case.dK, dK), ("dV", case.dV, dV)):
        g = got.float().cpu().numpy()
        assert rel_l2(g, want) <= TOL_RELL2_GRAD, name
        check_rows(name, g, want)
    ctx.close()
