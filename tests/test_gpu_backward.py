"""GPU: backward (dQ, dK, dV) and the partition driver against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import TOL_RELL2_GRAD, DeviceCase, check_forward, check_rows, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def run_partitioned(ctx, case):
    binding.peagle_attn_partitioned(ctx, case.prob, case.bparts, case.dQ_, case.dK_, case.dV_,
                                    case.ddO, case.O, case.LSE, case.dQ, case.dK, case.dV)
    assert binding.peagle_poll_status(ctx) == 0


def oracle_all(case):
    """Oracle O, LSE, dQ (full tensors) and dK, dV summed over the partitions."""
    w = case.w
    O = np.zeros((case.T, w.n_q_heads, w.head_dim))
    LSE = np.zeros((case.T, w.n_q_heads))
    dQ = np.zeros_like(O)
    dK = np.zeros((case.T, w.n_kv_heads, w.head_dim))
    dV = np.zeros_like(dK)
    for p in case.parts:
        sl = case.seq_slice(p["seq"])
        rows = np.arange(*p["q"])
        O[rows], LSE[rows] = case.oracle_fwd(p)
        dKs = np.zeros((sl.stop - sl.start, w.n_kv_heads, w.head_dim))
        dVs = np.zeros_like(dKs)
        dQ[rows], _, _ = case.oracle_bwd(p, dK=dKs, dV=dVs)
        dK[sl] += dKs
        dV[sl] += dVs
    return O, LSE, dQ, dK, dV


def check_grads(case, dQ, dK, dV):
    got = [t.float().cpu().numpy() for t in (case.dQ, case.dK, case.dV)]
    for name, g, want in zip(("dQ", "dK", "dV"), got, (dQ, dK, dV)):
        assert np.isfinite(g).all(), name
        assert rel_l2(g, want) <= TOL_RELL2_GRAD, (name, rel_l2(g, want))
        check_rows(name, g, want)


SMALL = [
    inputs.WORKLOADS["tiny"],
    inputs.Workload("d128_gqa", (200,), 3, 4, 2, 128, seed=3),
    inputs.Workload("ragged_segments", (333,), 4, 4, 2, 64, n_segments=3, seed=4),
    inputs.Workload("odd_group", (150,), 2, 3, 1, 64, seed=5),
    inputs.Workload("k1_causal", (300,), 1, 2, 2, 64, seed=6),
    inputs.Workload("two_seqs", (140, 70), 3, 2, 1, 64, n_segments=2, seed=7),
    inputs.Workload("d128_segments", (260,), 4, 8, 2, 128, n_segments=2, seed=8),
    inputs.Workload("many_tiles", (1100,), 2, 8, 1, 64, seed=13),        # > BWD_CQ query tiles per key tile
    # 20 depths: the deepest query tiles have more one-key-per-row chain tiles than the kernels
    # take pair by pair, the rest goes through the tensor-core path; 150 anchors: chain tiles
    # straddle two key tiles
    inputs.Workload("deep_chains", (150,), 20, 2, 1, 64, seed=14),
    # COD-subsampled metadata (retention 0.7): ragged depth blocks, chain tiles that are no
    # diagonals, Algorithm 1 on nested position sets
    inputs.Workload("cod_segments", (700,), 6, 4, 2, 64, n_segments=2, seed=15, cod_r=0.7),
    # a chain's tokens stored next to each other (depth-0 block, then anchor-major): the chain keys
    # fall into the query tile's own neighbourhood instead of one-key-per-row tiles
    inputs.Workload("anchor_major", (700,), 8, 4, 2, 64, n_segments=2, seed=17, order="anchor_major"),
    # more KV heads than the pair-by-pair kernels take: chain tiles stay on the tensor-core path
    inputs.Workload("many_kv_heads", (200,), 4, 24, 24, 64, seed=16),
]


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_partitioned_small_full_compare(ctx, w):
    case = DeviceCase(w)
    run_partitioned(ctx, case)
    O, LSE, dQ, dK, dV = oracle_all(case)
    check_forward(case.O.float().cpu().numpy(), case.LSE.t().cpu().numpy(), O, LSE)
    check_grads(case, dQ, dK, dV)


def test_partitioned_peaky_scores(ctx):
    case = DeviceCase(inputs.Workload("peaky", (400,), 4, 4, 1, 64, seed=9), q_std=1.0)
    run_partitioned(ctx, case)
    O, LSE, dQ, dK, dV = oracle_all(case)
    check_grads(case, dQ, dK, dV)


def test_bwd_adds_into_accumulators_and_partitions_sum_to_whole(ctx):
    """peagle_attn_fwd/bwd per partition with caller-owned fp32 accumulators: the sum over the
    partitions equals the unpartitioned oracle, and a second pass doubles it (ADD semantics)."""
    w = inputs.Workload("acc", (333,), 4, 4, 2, 64, n_segments=3, seed=4)
    case = DeviceCase(w)
    dK_acc = torch.zeros(case.T, w.n_kv_heads, w.head_dim, dtype=torch.float32, device="cuda")
    dV_acc = torch.zeros_like(dK_acc)
    for rep in range(2):
        for bp in case.bparts:
            binding.peagle_attn_fwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
            binding.peagle_attn_bwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.ddO,
                                    case.LSE, case.dQ, dK_acc, dV_acc)
        assert binding.peagle_poll_status(ctx) == 0
        whole = {"seq": 0, "q": (0, case.T), "k": [(0, case.T)]}
        dQ, dK, dV = case.oracle_bwd(whole)
        assert rel_l2(dK_acc.cpu().numpy(), (rep + 1) * dK) <= TOL_RELL2_GRAD
        assert rel_l2(dV_acc.cpu().numpy(), (rep + 1) * dV) <= TOL_RELL2_GRAD
        assert rel_l2(case.dQ.float().cpu().numpy(), dQ) <= TOL_RELL2_GRAD


def test_bwd_shuffled_token_order(ctx):
    w = inputs.Workload("shuffled", (100,), 4, 4, 2, 64, seed=10)
    anchor, depth = inputs.full_grid(100, 4)
    perm = np.random.default_rng(3).permutation(400)
    parts = [{"seq": 0, "q": (0, 400), "k": [(0, 400)]}]
    case = DeviceCase(w, anchor=anchor[perm], depth=depth[perm], cu=np.array([0, 400], np.int32),
                      parts=parts)
    run_partitioned(ctx, case)
    O, LSE, dQ, dK, dV = oracle_all(case)
    check_grads(case, dQ, dK, dV)


def test_bwd_rows_that_see_nothing_get_zero_gradients(ctx):
    w = inputs.Workload("subset", (90,), 3, 2, 1, 64, seed=11)
    anchor, depth = inputs.full_grid(90, 3)
    parts = [{"seq": 0, "q": (100, 200), "k": [(140, 160)]}]
    case = DeviceCase(w, anchor=anchor, depth=depth, cu=np.array([0, 270], np.int32), parts=parts)
    dK_acc = torch.zeros(270, 1, 64, dtype=torch.float32, device="cuda")
    dV_acc = torch.zeros_like(dK_acc)
    bp = case.bparts[0]
    binding.peagle_attn_fwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
    binding.peagle_attn_bwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.ddO,
                            case.LSE, case.dQ, dK_acc, dV_acc)
    assert binding.peagle_poll_status(ctx) == 0
    dQ, dK, dV = case.oracle_bwd(parts[0])
    got_dQ = case.dQ.float().cpu().numpy()
    assert np.isnan(got_dQ[:100]).all() and np.isnan(got_dQ[200:]).all()
    assert rel_l2(got_dQ[100:200], dQ) <= TOL_RELL2_GRAD
    empty = np.isneginf(case.LSE[:, 100:200].cpu().numpy()).T            # [rows][heads]
    assert empty.any() and np.all(got_dQ[100:200][empty] == 0)
    assert rel_l2(dK_acc.cpu().numpy(), dK) <= TOL_RELL2_GRAD
    assert rel_l2(dV_acc.cpu().numpy(), dV) <= TOL_RELL2_GRAD
    assert torch.all(dK_acc[:140] == 0) and torch.all(dK_acc[160:] == 0)


def full_size_checks(case, n_rows=16, n_keys=6, seed=0):
    """Checks that hold at any size, plus outputs the oracle can compute one by one."""
    w = case.w
    G = w.n_q_heads // w.n_kv_heads
    got_dQ, got_dK, got_dV = case.dQ.float(), case.dK.float(), case.dV.float()
    for t in (got_dQ, got_dK, got_dV):
        assert torch.isfinite(t).all()
    # (1) every row's probabilities sum to one, so  sum_k dV[k,g,:] = sum_{q, h in g} dO[q,h,:]
    want = case.ddO.float().view(case.T, w.n_kv_heads, G, w.head_dim).sum(dim=(0, 2))
    got = got_dV.sum(dim=0)
    assert rel_l2(got.cpu().numpy(), want.cpu().numpy()) <= TOL_RELL2_GRAD
    # (2) sum_k <dK[k,g], K[k,g]> = sum_{q, h in g} <dQ[q,h], Q[q,h]>  (both equal sum dS*S)
    lhs = (got_dK * case.dK_.float()).sum(dim=(0, 2))
    rhs = (got_dQ * case.dQ_.float()).view(case.T, w.n_kv_heads, G, w.head_dim).sum(dim=(0, 2, 3))
    scale = (got_dK.norm() * case.dK_.float().norm()).item()
    assert (lhs - rhs).abs().max().item() <= 2e-3 * scale
    # (3) sampled dQ rows
    rng = np.random.default_rng(seed)
    for p in case.parts:
        b, e = p["q"]
        rows = np.unique(np.concatenate([[b, e - 1], rng.integers(b, e, size=n_rows)]))
        dQ, _, _ = case.oracle_bwd(p, rows=rows)
        g = got_dQ[torch.as_tensor(rows, device="cuda")].cpu().numpy()
        assert rel_l2(g, dQ) <= TOL_RELL2_GRAD
        check_rows("dQ", g, dQ)
    # (4) dK / dV of keys few queries see: chain tokens (depth >= 1) and the last depth-0
    # tokens of a sequence; every query that sees them is evaluated by the oracle
    for s in range(len(case.cu) - 1):
        sl = case.seq_slice(s)
        a, d = case.anchor[sl], case.depth[sl]
        n = int(a.max()) + 1
        keys = np.concatenate([np.nonzero((d == 0) & (a >= n - 2))[0],
                               rng.choice(np.nonzero(d >= 1)[0], size=n_keys, replace=False)])
        need = np.zeros(sl.stop - sl.start, bool)
        for k in keys:
            if d[k] == 0:
                need |= a >= a[k]
            else:
                need |= (a == a[k]) & (d >= d[k])
        dKs = np.zeros((sl.stop - sl.start, w.n_kv_heads, w.head_dim))
        dVs = np.zeros_like(dKs)
        for p in case.parts:
            if p["seq"] != s:
                continue
            rows = np.nonzero(need)[0] + sl.start
            rows = rows[(rows >= p["q"][0]) & (rows < p["q"][1])]
            if rows.size:
                case.oracle_bwd(p, rows=rows, dK=dKs, dV=dVs)
        kt = torch.as_tensor(keys + sl.start, device="cuda")
        assert rel_l2(got_dK[kt].cpu().numpy(), dKs[keys]) <= TOL_RELL2_GRAD
        assert rel_l2(got_dV[kt].cpu().numpy(), dVs[keys]) <= TOL_RELL2_GRAD
        check_rows("dK", got_dK[kt].cpu().numpy(), dKs[keys])
        check_rows("dV", got_dV[kt].cpu().numpy(), dVs[keys])
        if s >= 2:
            break


@pytest.mark.parametrize("name", ["qwen3coder_n2048", "gptoss_n4096", "gptoss_n4096_anchor_major",
                                  "p90_n11008_s4"])
def test_partitioned_full_size(ctx, name):
    case = DeviceCase(inputs.WORKLOADS[name])
    run_partitioned(ctx, case)
    full_size_checks(case)


def test_partitioned_one_kv_group_in_full(ctx):
    """Config 2 restricted to its first KV group (all 8 query heads of it, every row): O, LSE,
    dQ of those heads and dK, dV of the group are compared in full."""
    w = inputs.WORKLOADS["qwen3coder_n2048"]
    case = DeviceCase(w)
    run_partitioned(ctx, case)
    G = w.n_q_heads // w.n_kv_heads
    p = case.parts[0]
    O, LSE = case.oracle_fwd(p, heads=(0, G))
    dQ, dK, dV = case.oracle_bwd(p, heads=(0, G))
    check_forward(case.O[:, :G].float().cpu().numpy(), case.LSE[:G].t().cpu().numpy(), O, LSE)
    assert rel_l2(case.dQ[:, :G].float().cpu().numpy(), dQ) <= TOL_RELL2_GRAD
    assert rel_l2(case.dK[:, 0].float().cpu().numpy(), dK[:, 0]) <= TOL_RELL2_GRAD
    assert rel_l2(case.dV[:, 0].float().cpu().numpy(), dV[:, 0]) <= TOL_RELL2_GRAD
    check_rows("dQ", case.dQ[:, :G].float().cpu().numpy(), dQ)
    check_rows("dK", case.dK[:, 0].float().cpu().numpy(), dK[:, 0])
    check_rows("dV", case.dV[:, 0].float().cpu().numpy(), dV[:, 0])


def test_headline_one_kv_group_in_full(ctx):
    """Config 3 (the headline shape) restricted to one KV group: O, LSE, dQ of its 8 query heads
    and dK, dV of the group, every row, whole-tensor norms and per-row bounds.  This is the path
    that only exists at full size: every early depth-0 key row is the sum of reductions from
    hundreds of work items."""
    w = inputs.WORKLOADS["gptoss_n4096"]
    case = DeviceCase(w)
    run_partitioned(ctx, case)
    G = w.n_q_heads // w.n_kv_heads
    g = 3
    hs = (g * G, (g + 1) * G)
    p = case.parts[0]
    O, LSE = case.oracle_fwd(p, heads=hs)
    dQ, dK, dV = case.oracle_bwd(p, heads=hs)
    check_forward(case.O[:, hs[0]:hs[1]].float().cpu().numpy(),
                  case.LSE[hs[0]:hs[1]].t().cpu().numpy(), O, LSE)
    got = {"dQ": case.dQ[:, hs[0]:hs[1]].float().cpu().numpy(),
           "dK": case.dK[:, g].float().cpu().numpy(), "dV": case.dV[:, g].float().cpu().numpy()}
    for name, want in (("dQ", dQ), ("dK", dK[:, g]), ("dV", dV[:, g])):
        assert rel_l2(got[name], want) <= TOL_RELL2_GRAD, name
        check_rows(name, got[name], want)


def test_longtail_varlen_batch(ctx):
    """Config 5: 17 sequences, 19 partitions; the shortest sequence is compared in full for one
    KV group, the rest through the size-independent checks on sampled rows."""
    w = inputs.WORKLOADS["longtail_varlen"]
    case = DeviceCase(w)
    run_partitioned(ctx, case)
    G = w.n_q_heads // w.n_kv_heads
    s = int(np.argmin(np.diff(case.cu)))
    p = [q for q in case.parts if q["seq"] == s][0]
    sl = case.seq_slice(s)
    O, LSE = case.oracle_fwd(p, heads=(0, G))
    dQ, dK, dV = case.oracle_bwd(p, heads=(0, G))
    check_forward(case.O[sl, :G].float().cpu().numpy(), case.LSE[:G, sl].t().cpu().numpy(), O, LSE)
    assert rel_l2(case.dQ[sl, :G].float().cpu().numpy(), dQ) <= TOL_RELL2_GRAD
    assert rel_l2(case.dK[sl, 0].float().cpu().numpy(), dK[:, 0]) <= TOL_RELL2_GRAD
    assert rel_l2(case.dV[sl, 0].float().cpu().numpy(), dV[:, 0]) <= TOL_RELL2_GRAD
    full_size_checks(case, n_rows=3, n_keys=3)
    # O / LSE of the two sequences that are split into two partitions, sampled rows of each part
    rng = np.random.default_rng(1)
    split = [q for q in case.parts if sum(1 for r in case.parts if r["seq"] == q["seq"]) > 1]
    assert len(split) == 4
    for p in split:
        b, e = p["q"]
        rows = np.unique(np.concatenate([[b, e - 1], rng.integers(b, e, size=6)]))
        O, LSE = case.oracle_fwd(p, rows=rows)
        rt = torch.as_tensor(rows, device="cuda")
        check_forward(case.O[rt].float().cpu().numpy(), case.LSE[:, rt].t().cpu().numpy(), O, LSE)


@pytest.mark.parametrize("w,shuffle", [
    (inputs.Workload("host", (333,), 4, 4, 2, 64, n_segments=3, seed=4), False),
    # several 2,048-row slices per partition, two sequences
    (inputs.Workload("host_slices", (1500, 700), 4, 4, 2, 64, n_segments=2, seed=5), False),
    # a token order in which keys sit after their queries, several slices
    (inputs.Workload("host_shuffled", (1300,), 4, 4, 2, 64, seed=6), True),
], ids=["one_slice", "many_slices", "shuffled"])
def test_host_entry_point_matches_device_entry_point(ctx, w, shuffle):
    if shuffle:
        cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
        perm = np.random.default_rng(7).permutation(anchor.shape[0])
        case = DeviceCase(w, anchor=anchor[perm], depth=depth[perm], cu=cu, parts=parts)
    else:
        case = DeviceCase(w)
    run_partitioned(ctx, case)
    hp = binding.Problem(case.cu, case.anchor, case.depth, w.K, w.n_q_heads, w.n_kv_heads,
                         w.head_dim, w.scale)
    outs = [torch.empty_like(t, device="cpu").pin_memory()
            for t in (case.O, case.LSE, case.dQ, case.dK, case.dV)]
    ins = [t.contiguous().pin_memory() for t in (case.Q, case.K, case.V, case.dO)]
    binding.peagle_attn_partitioned_host(ctx, hp, case.bparts, ins[0], ins[1], ins[2], ins[3],
                                         outs[0], outs[1], outs[2], outs[3], outs[4])
    O, LSE, dQ, dK, dV = oracle_all(case)
    check_forward(outs[0].float().numpy(), outs[1].t().numpy(), O, LSE)
    assert rel_l2(outs[2].float().numpy(), dQ) <= TOL_RELL2_GRAD
    assert rel_l2(outs[3].float().numpy(), dK) <= TOL_RELL2_GRAD
    assert rel_l2(outs[4].float().numpy(), dV) <= TOL_RELL2_GRAD
    assert torch.equal(outs[0], case.O.cpu())          # forward is deterministic
