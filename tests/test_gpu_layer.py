"""GPU: the layer slice run segment by segment (peagle_layer_partitioned: projection GEMMs, rotary
prologue, attention forward and backward per segment, dX / dW summed over the segments) against the
fp64 oracle of the same chain, through the C ABI.

Tolerances.  The GPU chain rounds to bf16 at every interface the layer has (fused rows, Q / K / V,
probabilities, O, dQ / dK / dV, the fused-row gradient, dX / dW), the oracle nowhere.  A bf16
rounding is a relative error of at most 2^-9 (rms 2^-9 / sqrt(3) = 1.1e-3); six to eight of them in
a row, independent, give 3e-3 to 4e-3 rms on the linear parts, and the rounding of Q and K moves
every score by about 2e-3 |s|, which the softmax passes on to O and to dS.  Bounds: O relative L2
<= 1e-2 and max-abs <= 3e-2, LSE max-abs <= 2e-2, dX and dW relative L2 <= 2e-2."""
import math

import numpy as np
import pytest
import torch

from oracle import layer_oracle as lo
from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import rel_l2

pytestmark = pytest.mark.gpu
ROPE_BASE = 500000.0


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def run_layer(ctx, w, d_model, parts_override=None):
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    if parts_override is not None:
        parts = parts_override(cu)
    T = int(cu[-1])
    X, W, dO = inputs.make_layer_tensors(T, d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seed)
    dev = torch.device("cuda:0")
    nan = float("nan")
    O = torch.full((T, w.n_q_heads, w.head_dim), nan, dtype=torch.bfloat16, device=dev)
    LSE = torch.full((w.n_q_heads, T), nan, dtype=torch.float32, device=dev)
    dX = torch.full((T, d_model), nan, dtype=torch.bfloat16, device=dev)
    dW = torch.full(tuple(W.shape), nan, dtype=torch.bfloat16, device=dev)
    prob = binding.Problem(cu, torch.from_numpy(anchor).to(dev), torch.from_numpy(depth).to(dev), w.K,
                           w.n_q_heads, w.n_kv_heads, w.head_dim, w.scale)
    bparts = [binding.Partition(p["seq"], p["q"], p["k"]) for p in parts]
    binding.peagle_layer_partitioned(ctx, prob, bparts, X.to(dev), W.to(dev), ROPE_BASE, dO.to(dev), O,
                                     LSE, dX, dW)
    assert binding.peagle_poll_status(ctx) == 0
    return dict(anchor=anchor, depth=depth, parts=parts, X=X, W=W, dO=dO, O=O, LSE=LSE, dX=dX, dW=dW, T=T)


def check_against_oracle(w, r):
    want = lo.layer_segmented(r["X"].double().numpy(), r["W"].double().numpy(), r["anchor"], r["depth"],
                              w.n_q_heads, w.n_kv_heads, w.head_dim, ROPE_BASE, w.scale,
                              r["dO"].double().numpy(), r["parts"])
    O, LSE = r["O"].float().cpu().numpy(), r["LSE"].t().cpu().numpy()
    dX, dW = r["dX"].float().cpu().numpy(), r["dW"].float().cpu().numpy()
    for t in (O, LSE, dX, dW):
        assert np.isfinite(t).all()
    errs = (rel_l2(O, want[0]), float(np.abs(O - want[0]).max()), float(np.abs(LSE - want[1]).max()),
            rel_l2(dX, want[2]), rel_l2(dW, want[3]))
    print("layer errors O rel / O max / LSE max / dX rel / dW rel:", errs)
    assert errs[0] <= 1e-2 and errs[1] <= 3e-2 and errs[2] <= 2e-2 and errs[3] <= 2e-2 and errs[4] <= 2e-2
    return errs


@pytest.mark.parametrize("w,d_model", [
    (inputs.Workload("layer_small", (150,), 4, 4, 2, 64, n_segments=3, seed=31), 128),
    # ragged everything: d_model not a multiple of the k slab, segment blocks not tile aligned
    (inputs.Workload("layer_ragged", (333,), 3, 6, 2, 64, n_segments=2, seed=32), 200),
    (inputs.Workload("layer_d128", (260,), 4, 8, 2, 128, n_segments=2, seed=33), 192),
    (inputs.Workload("layer_two_seqs", (140, 90), 3, 4, 1, 64, n_segments=2, seed=34), 64),
    (inputs.Workload("layer_medium", (1024,), 4, 8, 2, 64, n_segments=3, seed=35), 256),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_segmented_layer_matches_oracle(ctx, w, d_model):
    check_against_oracle(w, run_layer(ctx, w, d_model))


def test_p90_shape_segmented_equals_single_pass_and_sampled_forward(ctx):
    """The P90-length configuration's segmentation (n = 11,008 in four segments; the layer is taken
    narrower -- 8 / 2 heads, d_model 512 -- so that the oracle's share stays in seconds): the
    segmented run equals a single pass over the whole sequence on the GPU (Section 3.2's identity,
    at bf16 accuracy), and O / LSE of sampled rows equal the oracle's."""
    w = inputs.Workload("layer_p90", (11008,), 8, 8, 2, 64, n_segments=4, seed=36)
    seg = run_layer(ctx, w, 512)
    whole = run_layer(ctx, w, 512, parts_override=lambda cu: [{"seq": 0, "q": (0, int(cu[-1])), "k": [(0, int(cu[-1]))]}])
    assert rel_l2(seg["O"].float().cpu().numpy(), whole["O"].float().cpu().numpy()) <= 2e-3
    assert rel_l2(seg["dX"].float().cpu().numpy(), whole["dX"].float().cpu().numpy()) <= 1e-2
    assert rel_l2(seg["dW"].float().cpu().numpy(), whole["dW"].float().cpu().numpy()) <= 1e-2
    # sampled rows of the last segment against the oracle: its keys are recomputed depth-0 rows
    p = seg["parts"][-1]
    rows = np.unique(np.concatenate([[p["q"][0], p["q"][1] - 1],
                                     np.random.default_rng(0).integers(p["q"][0], p["q"][1], size=16)]))
    vis = np.concatenate([np.arange(b, e) for b, e in p["k"]])
    X, W = seg["X"].double().numpy(), seg["W"].double().numpy()
    from oracle import rope_oracle as ro
    Q, K, V = ro.rope_qkv_fwd(X[vis] @ W.T, seg["anchor"][vis], seg["depth"][vis], 8, 2, 64, ROPE_BASE)
    local = np.searchsorted(vis, rows)
    O, LSE, _, _, _ = lo.attention_np(seg["anchor"][vis], seg["depth"][vis], Q, K, V,
                                      np.zeros((len(rows), 8, 64)), w.scale, local)
    rt = torch.as_tensor(rows, device="cuda")
    gO, gL = seg["O"][rt].float().cpu().numpy(), seg["LSE"][:, rt].t().cpu().numpy()
    assert rel_l2(gO, O) <= 1e-2 and np.abs(gL - LSE).max() <= 2e-2
