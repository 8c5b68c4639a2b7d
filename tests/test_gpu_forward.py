"""GPU: forward (O, LSE) of the CUDA path against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import DeviceCase, check_forward

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def run_fwd_all(ctx, case):
    for bp in case.bparts:
        binding.peagle_attn_fwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
    assert binding.peagle_poll_status(ctx) == 0


def compare_rows(case, part, rows, heads=None):
    want_O, want_LSE = case.oracle_fwd(part, rows=rows, heads=heads)
    h0, h1 = (0, case.w.n_q_heads) if heads is None else heads
    rows_t = torch.as_tensor(np.asarray(rows), device="cuda")
    got_O = case.O[rows_t][:, h0:h1].float().cpu().numpy()
    got_LSE = case.LSE[h0:h1][:, rows_t].t().cpu().numpy()
    check_forward(got_O, got_LSE, want_O, want_LSE)


SMALL = [
    inputs.WORKLOADS["tiny"],                                             # cfg 1
    inputs.Workload("d128_gqa", (200,), 3, 4, 2, 128, seed=3),            # head_dim 128, ragged tail
    inputs.Workload("ragged_segments", (333,), 4, 4, 2, 64, n_segments=3, seed=4),
    inputs.Workload("odd_group", (150,), 2, 3, 1, 64, seed=5),            # one head per CTA
    inputs.Workload("k1_causal", (300,), 1, 2, 2, 64, seed=6),            # plain causal attention
    inputs.Workload("two_seqs", (140, 70), 3, 2, 1, 64, n_segments=2, seed=7),
    inputs.Workload("d128_segments", (260,), 4, 8, 2, 128, n_segments=2, seed=8),
    # 20 depths: the deepest query tiles have more one-key-per-row chain tiles than the kernels
    # take pair by pair, the rest goes through the tensor-core path; 150 anchors: chain tiles
    # straddle two key tiles
    inputs.Workload("deep_chains", (150,), 20, 2, 1, 64, seed=14),
    # COD-subsampled metadata (retention 0.7): ragged depth blocks, chain tiles that are no
    # diagonals, Algorithm 1 on nested position sets
    inputs.Workload("cod_segments", (700,), 6, 4, 2, 64, n_segments=2, seed=15, cod_r=0.7),
    # more KV heads than the pair-by-pair kernels take: chain tiles stay on the tensor-core path
    inputs.Workload("many_kv_heads", (200,), 4, 24, 24, 64, seed=16),
    inputs.Workload("anchor_major", (700,), 8, 4, 2, 64, n_segments=2, seed=17, order="anchor_major"),
]


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_forward_small_full_compare(ctx, w):
    case = DeviceCase(w)
    run_fwd_all(ctx, case)
    for p in case.parts:
        compare_rows(case, p, np.arange(*p["q"]))


def test_forward_peaky_scores_exercise_rescaling(ctx):
    case = DeviceCase(inputs.Workload("peaky", (400,), 4, 4, 1, 64, seed=9), q_std=1.0)
    run_fwd_all(ctx, case)
    for p in case.parts:
        compare_rows(case, p, np.arange(*p["q"]))


def test_forward_shuffled_token_order(ctx):
    w = inputs.Workload("shuffled", (100,), 4, 4, 2, 64, seed=10)
    anchor, depth = inputs.full_grid(100, 4)
    perm = np.random.default_rng(3).permutation(400)
    anchor, depth = anchor[perm], depth[perm]
    parts = [{"seq": 0, "q": (0, 400), "k": [(0, 400)]}]
    case = DeviceCase(w, anchor=anchor, depth=depth, cu=np.array([0, 400], np.int32), parts=parts)
    run_fwd_all(ctx, case)
    compare_rows(case, parts[0], np.arange(400))


def test_forward_partition_writes_only_its_rows_and_handles_empty_rows(ctx):
    w = inputs.Workload("subset", (90,), 3, 2, 1, 64, seed=11)
    anchor, depth = inputs.full_grid(90, 3)
    # rows 100..199 with only tokens 40..149 visible: depth-0 rows of anchors < 40 do not occur,
    # but chain rows whose own depth-0 context is cut still see something; rows 150.. see keys
    # only through the range, some rows end up with an empty set
    parts = [{"seq": 0, "q": (100, 200), "k": [(140, 160)]}]
    case = DeviceCase(w, anchor=anchor, depth=depth, cu=np.array([0, 270], np.int32), parts=parts)
    run_fwd_all(ctx, case)
    O = case.O.float().cpu().numpy()
    assert np.isnan(O[:100]).all() and np.isnan(O[200:]).all()      # untouched (poisoned) rows
    compare_rows(case, parts[0], np.arange(100, 200))
    lse = case.LSE[:, 100:200].cpu().numpy()
    assert np.isneginf(lse).any()                                   # some rows see nothing


def test_forward_no_visible_keys_at_all(ctx):
    w = inputs.Workload("nokeys", (20,), 2, 2, 1, 64, seed=12)
    anchor, depth = inputs.full_grid(20, 2)
    parts = [{"seq": 0, "q": (0, 20), "k": [(30, 40)]}]             # depth-1 keys of later anchors
    case = DeviceCase(w, anchor=anchor, depth=depth, cu=np.array([0, 40], np.int32), parts=parts)
    run_fwd_all(ctx, case)
    assert torch.all(case.O[:20] == 0) and torch.isneginf(case.LSE[:, :20]).all()


@pytest.mark.parametrize("name", ["qwen3coder_n2048", "gptoss_n4096", "p90_n11008_s4"])
def test_forward_full_size_sampled_rows(ctx, name):
    """Full-size launch; rows sampled from every partition (first/last tiles, ragged tail,
    random interior) are compared with the oracle one by one."""
    case = DeviceCase(inputs.WORKLOADS[name])
    run_fwd_all(ctx, case)
    assert not torch.isnan(case.O.float()).any()
    rng = np.random.default_rng(0)
    for p in case.parts:
        b, e = p["q"]
        rows = np.unique(np.concatenate([np.arange(b, b + 3), np.arange(e - 3, e),
                                         rng.integers(b, e, size=18)]))
        compare_rows(case, p, rows)
