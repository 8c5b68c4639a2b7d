"""CPU pins of the segmented-layer oracle (projection -> rotary -> masked attention and the
gradients of <O, dO>): its attention against the C oracle, the whole chain against an independent
torch formulation with autograd, central finite differences, and Section 3.2's identity
"segment by segment with gradient accumulation = the whole sequence at once"."""
import math

import numpy as np
import pytest
import torch

from oracle import layer_oracle as lo
from oracle import partition as opart
from oracle import peagle_oracle as orc
from paper_2602_01469_b200 import inputs


def oracle_assign(anchor, depth, K, bounds):
    P = inputs.position_sets(anchor, depth, K)
    A, _, _ = opart.assign_segments(P, len(bounds) - 1, bounds[-1], B=bounds)
    return np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)


def make_layer(w, d_model, seed):
    cu, anchor, depth, parts = inputs.build_case(w, oracle_assign)
    T = int(cu[-1])
    X, W, dO = inputs.make_layer_tensors(T, d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, seed)
    return anchor, depth, parts, X.double().numpy(), W.double().numpy(), dO.double().numpy()


def test_numpy_attention_equals_the_c_oracle():
    w = inputs.Workload("a", (37,), 4, 4, 2, 16, n_segments=2, seed=3)
    cu, anchor, depth, parts = inputs.build_case(w, oracle_assign)
    T = int(cu[-1])
    Q, K, V, dO = inputs.make_tensors(T, 4, 2, 16, seed=3, q_std=1.0)
    perm = np.random.default_rng(2).permutation(T)          # the mask depends on metadata only
    anchor, depth = anchor[perm], depth[perm]
    rows = np.sort(np.random.default_rng(3).choice(T, size=50, replace=False))
    O, LSE, dQ, dK, dV = lo.attention_np(anchor, depth, Q.double().numpy(), K.double().numpy(),
                                         V.double().numpy(), dO.double().numpy()[rows], 0.3, rows, block=16)
    wO, wL = orc.attn_fwd(anchor, depth, Q, K, V, 0.3, rows=rows)
    wdQ, wdK, wdV = orc.attn_bwd(anchor, depth, Q, K, V, dO, 0.3, rows=rows)
    for got, want in ((O, wO), (LSE, wL), (dQ, wdQ), (dK, wdK), (dV, wdV)):
        assert np.allclose(got, want, atol=1e-12)


def torch_chain(X, W, anchor, depth, Hq, Hkv, D, base, scale, dO):
    """The same chain written independently with torch ops; gradients by autograd."""
    x = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    w = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    T = x.shape[0]
    qkv = x @ w.t()
    pos = torch.tensor(anchor + depth, dtype=torch.float64)
    inv = torch.tensor([base ** (-2.0 * i / D) for i in range(D // 2)], dtype=torch.float64)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]

    def rot(t):                                     # LLaMA's rotate-half form
        lo_, hi_ = t[..., : D // 2], t[..., D // 2:]
        return torch.cat([lo_ * cos - hi_ * sin, hi_ * cos + lo_ * sin], dim=-1)

    q = rot(qkv[:, : Hq * D].reshape(T, Hq, D))
    k = rot(qkv[:, Hq * D:(Hq + Hkv) * D].reshape(T, Hkv, D))
    v = qkv[:, (Hq + Hkv) * D:].reshape(T, Hkv, D)
    M = torch.tensor(orc.mask_dense(anchor, depth).astype(bool))
    kx, vx = k.repeat_interleave(Hq // Hkv, 1), v.repeat_interleave(Hq // Hkv, 1)
    S = torch.einsum("qhd,khd->hqk", q, kx) * scale
    S = S.masked_fill(~M[None], float("-inf"))
    O = torch.einsum("hqk,khd->qhd", torch.softmax(S, dim=-1), vx)
    (O * torch.tensor(dO)).sum().backward()
    return O.detach().numpy(), torch.logsumexp(S, -1).t().detach().numpy(), x.grad.numpy(), w.grad.numpy()


def test_whole_chain_equals_torch_autograd():
    w = inputs.Workload("c", (13,), 3, 4, 2, 8, seed=5)
    anchor, depth, parts, X, W, dO = make_layer(w, 24, seed=5)
    got = lo.layer_whole(X, W, anchor, depth, 4, 2, 8, 10000.0, 0.35, dO)
    want = torch_chain(X, W, anchor, depth, 4, 2, 8, 10000.0, 0.35, dO)
    for g, t in zip(got, want):
        assert np.allclose(g, t, atol=1e-11)


def test_chain_gradients_by_central_differences():
    w = inputs.Workload("f", (6,), 3, 2, 1, 4, n_segments=2, seed=6)
    anchor, depth, parts, X, W, dO = make_layer(w, 8, seed=6)
    args = (anchor, depth, 2, 1, 4, 500000.0, 0.5)
    _, _, dX, dW = lo.layer_segmented(X, W, *args, dO, parts)

    def loss(Xp, Wp):
        O, _, _, _ = lo.layer_whole(Xp, Wp, *args, dO)
        return float((O * dO).sum())

    rng = np.random.default_rng(0)
    eps = 1e-6
    for which, grad in ((0, dX), (1, dW)):
        for idx in rng.choice(grad.size, size=20, replace=False):
            up, dn = [X.copy(), W.copy()], [X.copy(), W.copy()]
            up[which].reshape(-1)[idx] += eps
            dn[which].reshape(-1)[idx] -= eps
            fd = (loss(*up) - loss(*dn)) / (2 * eps)
            assert fd == pytest.approx(grad.reshape(-1)[idx], rel=1e-6, abs=1e-8)


@pytest.mark.parametrize("case", ["three_segments", "two_sequences_shape", "cod"])
def test_segment_by_segment_equals_the_whole_sequence(case):
    """Section 3.2: a separate forward-backward pass per segment with recomputed depth-0 K / V and
    accumulated gradients gives the gradients of the whole sequence."""
    if case == "three_segments":
        w = inputs.Workload("s3", (41,), 4, 4, 2, 8, n_segments=3, seed=7)
    elif case == "two_sequences_shape":
        w = inputs.Workload("s4", (30,), 8, 4, 4, 16, n_segments=4, seed=8)
    else:
        w = inputs.Workload("sc", (50,), 5, 2, 1, 8, n_segments=3, seed=9, cod_r=0.7)
    anchor, depth, parts, X, W, dO = make_layer(w, 40, seed=11)
    assert len(parts) == w.n_segments
    args = (anchor, depth, w.n_q_heads, w.n_kv_heads, w.head_dim, 500000.0, 1 / math.sqrt(w.head_dim))
    whole = lo.layer_whole(X, W, *args, dO)
    seg = lo.layer_segmented(X, W, *args, dO, parts)
    for a, b in zip(seg, whole):
        assert np.allclose(a, b, atol=1e-11)
    # a depth-0 token of the first segment collects dX from every later segment that sees it
    later_only = lo.layer_segmented(X, W, *args, dO, parts[1:])[2]
    first_d0 = np.arange(*parts[0]["q"])[depth[parts[0]["q"][0]:parts[0]["q"][1]] == 0]
    assert np.abs(later_only[first_d0]).max() > 0
