"""GPU: the device predicate and the tile classifier against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import peagle_oracle as orc
from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import DeviceCase, check_forward

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def device_problem(cu, anchor, depth, K, Hq=2, Hkv=1, D=64):
    d_a = torch.from_numpy(np.ascontiguousarray(anchor)).cuda()
    d_d = torch.from_numpy(np.ascontiguousarray(depth)).cuda()
    return binding.Problem(cu, d_a, d_d, K, Hq, Hkv, D, 0.125)


@pytest.mark.parametrize("n,K,shuffle", [(8, 4, False), (37, 3, True), (130, 2, True)])
def test_mask_dense_matches_oracle(ctx, n, K, shuffle):
    anchor, depth = inputs.full_grid(n, K)
    if shuffle:
        perm = np.random.default_rng(n).permutation(n * K)
        anchor, depth = anchor[perm], depth[perm]
    T = n * K
    prob = device_problem([0, T], anchor, depth, K)
    got = binding.peagle_mask_dense(ctx, prob, binding.Partition(0, (0, T)))
    assert np.array_equal(got, orc.mask_dense(anchor, depth))
    # a partition: rows 5..T-3, two visible ranges
    kr = [(0, T // 3), (T // 2, T - 1)]
    got = binding.peagle_mask_dense(ctx, prob, binding.Partition(0, (5, T - 3), kr))
    want = orc.mask_dense(anchor, depth)[5:T - 3].copy()
    vis = np.zeros(T, bool)
    for b, e in kr:
        vis[b:e] = True
    want[:, ~vis] = 0
    assert np.array_equal(got, want)
    assert binding.peagle_poll_status(ctx) == 0


def test_mask_dense_two_sequences(ctx):
    a1, d1 = inputs.full_grid(9, 3)
    a2, d2 = inputs.full_grid(5, 3)
    anchor, depth = np.concatenate([a1, a2]), np.concatenate([d1, d2])
    prob = device_problem([0, 27, 42], anchor, depth, 3)
    got = binding.peagle_mask_dense(ctx, prob, binding.Partition(1, (27, 42)))
    assert got[:, :27].sum() == 0
    assert np.array_equal(got[:, 27:], orc.mask_dense(a2, d2))


def fig3_tokens():
    P = [[0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15], [1, 3, 4, 6, 7, 9, 10, 12, 14, 15],
         [2, 5, 7, 8, 11, 13, 15], [3, 6, 9, 12, 14]]          # Section 3.2 worked example
    anchor = np.array([p - g for g, ps in enumerate(P) for p in ps], np.int32)
    depth = np.array([g for g, ps in enumerate(P) for _ in ps], np.int32)
    return anchor, depth


def test_mask_dense_cod_example(ctx):
    anchor, depth = fig3_tokens()
    prob = device_problem([0, 38], anchor, depth, 4)
    got = binding.peagle_mask_dense(ctx, prob, binding.Partition(0, (0, 38)))
    assert got.sum() == 344
    assert np.array_equal(got, orc.mask_dense(anchor, depth))


@pytest.mark.parametrize("name", ["tiny", "qwen3coder_n2048", "gptoss_n4096", "p90_n11008_s4"])
def test_tile_classes_match_oracle_on_workloads(ctx, name):
    w = inputs.WORKLOADS[name]
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    prob = device_problem(cu, anchor, depth, w.K, w.n_q_heads, w.n_kv_heads, w.head_dim)
    bm, bn = binding.peagle_tile_shape(ctx, w.head_dim)
    for p in parts:
        got = binding.peagle_classify_tiles(ctx, prob, binding.Partition(p["seq"], p["q"], p["k"]))
        want, _, _ = orc.classify_tiles(anchor, depth, p["q"][0], p["q"][1], p["k"], bm, bn)
        assert got.shape == want.shape
        assert np.array_equal(got, want)
    if name == "gptoss_n4096":     # 128x128 tiles, depth-major: closed-form counts
        assert int((got == 2).sum()) == 8 * 32 * 31 // 2 == 3968
        assert int((got == 1).sum()) == 8 * 32 + 32 * 8 * 7 // 2 == 1152
    assert binding.peagle_poll_status(ctx) == 0


def test_tile_classes_longtail_sequences(ctx):
    w = inputs.WORKLOADS["longtail_varlen"]
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    prob = device_problem(cu, anchor, depth, w.K, w.n_q_heads, w.n_kv_heads, w.head_dim)
    assert len(parts) == 19            # 17 sequences, two of them longer than 8,192 tokens
    for p in parts:
        if p["seq"] not in (6, 7, 12):  # the two split sequences and the shortest one
            continue
        sl = slice(int(cu[p["seq"]]), int(cu[p["seq"] + 1]))
        off = sl.start
        got = binding.peagle_classify_tiles(ctx, prob, binding.Partition(p["seq"], p["q"], p["k"]))
        want, _, _ = orc.classify_tiles(anchor[sl], depth[sl], p["q"][0] - off, p["q"][1] - off,
                                        [(b - off, e - off) for b, e in p["k"]], 128, 128)
        assert np.array_equal(got, want)


def test_tile_classes_shuffled_and_cod(ctx):
    anchor, depth = inputs.full_grid(300, 4)
    perm = np.random.default_rng(5).permutation(1200)
    anchor, depth = anchor[perm], depth[perm]
    prob = device_problem([0, 1200], anchor, depth, 4)
    part = binding.Partition(0, (17, 1100), [(3, 500), (640, 1199)])
    got = binding.peagle_classify_tiles(ctx, prob, part)
    want, _, _ = orc.classify_tiles(anchor, depth, 17, 1100, [(3, 500), (640, 1199)], 128, 128)
    assert np.array_equal(got, want)
    a, d = fig3_tokens()
    prob = device_problem([0, 38], a, d, 4)
    got = binding.peagle_classify_tiles(ctx, prob, binding.Partition(0, (0, 38)))
    want, _, _ = orc.classify_tiles(a, d, 0, 38, None, 128, 128)
    assert np.array_equal(got, want)


def test_bad_metadata_is_reported_not_fatal(ctx):
    anchor, depth = inputs.full_grid(10, 2)
    depth = depth.copy()
    depth[3] = 2                     # depth >= K
    prob = device_problem([0, 20], anchor, depth, 2)
    binding.peagle_classify_tiles(ctx, prob, binding.Partition(0, (0, 20)))
    assert binding.peagle_poll_status(ctx) == binding.STATUS["BAD_META"]
    assert binding.peagle_poll_status(ctx) == 0       # cleared by the poll


def test_argument_errors(ctx):
    anchor, depth = inputs.full_grid(10, 2)
    prob = device_problem([0, 20], anchor, depth, 2)
    S = binding.STATUS

    def status_of(fn):
        with pytest.raises(binding.PeagleError) as e:
            fn()
        return e.value.status

    P = binding.Partition
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, prob, P(1, (0, 20)))) == S["BAD_RANGE"]
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, prob, P(0, (5, 21)))) == S["BAD_RANGE"]
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, prob, P(0, (7, 5)))) == S["BAD_RANGE"]
    assert status_of(lambda: binding.peagle_classify_tiles(
        ctx, prob, P(0, (0, 20), [(5, 10), (8, 12)]))) == S["BAD_RANGE"]
    assert status_of(lambda: binding.peagle_classify_tiles(
        ctx, prob, P(0, (0, 20), [(5, 5)]))) == S["BAD_RANGE"]
    assert status_of(lambda: binding.peagle_classify_tiles(
        ctx, prob, P(0, (0, 20), [(i, i + 1) for i in range(0, 20, 2)] * 4))) in (S["BAD_RANGE"], S["TOO_LARGE"])
    bad = binding.Problem([0, 20], prob.anchor, prob.depth, 2, 3, 2, 64, 0.125)
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, bad, P(0, (0, 20)))) == S["BAD_SHAPE"]
    bad = binding.Problem([0, 20], prob.anchor, prob.depth, 2, 2, 1, 96, 0.125)
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, bad, P(0, (0, 20)))) == S["BAD_SHAPE"]
    bad = binding.Problem([0, 19], prob.anchor, prob.depth, 300, 2, 1, 64, 0.125)
    assert status_of(lambda: binding.peagle_classify_tiles(ctx, bad, P(0, (0, 19)))) == S["BAD_SHAPE"]
    # empty query range is a no-op
    assert binding.peagle_classify_tiles(ctx, prob, P(0, (4, 4))).shape[0] == 0


def test_bounded_wait_runs_out_and_reports_timeout():
    """The expiry path of the kernels' waits, made to happen on the host's terms: a barrier nothing
    arrives at, a 20 ms limit.  The kernel returns, the status word says TIMEOUT once, and the
    context goes on working (a forward after it matches the oracle)."""
    import time
    c = binding.Context(0)
    try:
        t0 = time.perf_counter()
        binding.peagle_selftest_wait_expiry(c, 20)
        assert 0.015 <= time.perf_counter() - t0 < 5.0
        assert binding.peagle_poll_status(c) == binding.STATUS["TIMEOUT"]
        assert binding.peagle_poll_status(c) == 0                      # reported once, then cleared
        case = DeviceCase(inputs.WORKLOADS["tiny"])
        binding.peagle_attn_fwd(c, case.prob, case.bparts[0], case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
        assert binding.peagle_poll_status(c) == 0
        O, LSE = case.oracle_fwd(case.parts[0])
        check_forward(case.O.float().cpu().numpy(), case.LSE.t().cpu().numpy(), O, LSE)
    finally:
        c.close()
