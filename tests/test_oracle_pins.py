"""Pins of the fp64 CPU oracle to things other than itself: sets listed by hand from the
paper's prose, the printed worked example, closed forms, library causal attention, autograd
and finite differences.  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import partition as opart
from oracle import peagle_oracle as orc
from paper_2602_01469_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- helpers (independent)
def chain_set(a, d):
    """What a drafter anchored at real token a sees when it predicts depth d (Section 2,
    parallel drafting): real tokens 0..a, then its own mask-token positions 1..d."""
    return {(j, 0) for j in range(a + 1)} | {(a, e) for e in range(1, d + 1)}


def dense_from_sets(anchor, depth):
    tok = {(int(a), int(d)): i for i, (a, d) in enumerate(zip(anchor, depth))}
    M = np.zeros((len(anchor), len(anchor)), np.uint8)
    for (a, d), q in tok.items():
        for key in chain_set(a, d):
            if key in tok:
                M[q, tok[key]] = 1
    return M


def read_fig3():
    P, total = [], None
    for line in open(os.path.join(GOLD, "fig3_cod_example.txt")):
        if line.startswith("depth"):
            P.append([int(x) for x in line.split(":")[1].split()])
        elif line.startswith("total"):
            total = int(line.split(":")[1])
    return P, total


def fig3_tokens():
    P, _ = read_fig3()
    anchor = np.array([p - g for g, ps in enumerate(P) for p in ps], np.int32)
    depth = np.array([g for g, ps in enumerate(P) for _ in ps], np.int32)
    return P, anchor, depth


def rand_case(n, K, Hq, Hkv, D, seed, std=None):
    anchor, depth = inputs.full_grid(n, K)
    Q, Kt, V, dO = inputs.make_tensors(n * K, Hq, Hkv, D, seed, q_std=std)
    return anchor, depth, Q, Kt, V, dO


def torch_dense_attention(M, Q, K, V, scale):
    """softmax(scale QK^T + mask) V in fp64 with torch ops, GQA expanded; returns O [T,Hq,D], LSE [T,Hq]."""
    Hq, Hkv = Q.shape[1], K.shape[1]
    Kx = K.repeat_interleave(Hq // Hkv, dim=1)
    Vx = V.repeat_interleave(Hq // Hkv, dim=1)
    S = torch.einsum("qhd,khd->hqk", Q, Kx) * scale
    S = S.masked_fill(~torch.as_tensor(M, dtype=torch.bool)[None], float("-inf"))
    lse = torch.logsumexp(S, dim=-1)
    O = torch.einsum("hqk,khd->qhd", torch.softmax(S, dim=-1), Vx)
    return O, lse.transpose(0, 1)


# ---------------------------------------------------------------- mask
def test_mask_hand_listed_n3_k3():
    want = {}
    for line in open(os.path.join(GOLD, "mask_n3_k3.txt")):
        if line.startswith("#") or not line.strip():
            continue
        q, ks = line.split(":")
        want[tuple(map(int, q.split(",")))] = {tuple(map(int, k.split(","))) for k in ks.split()}
    assert len(want) == 9
    toks = [(a, d) for d in range(3) for a in range(3)]
    for (aq, dq) in toks:
        got = {(ak, dk) for (ak, dk) in toks if orc.allowed(aq, dq, ak, dk)}
        assert got == want[(aq, dq)], (aq, dq)


@pytest.mark.parametrize("n,K", [(1, 1), (5, 1), (8, 4), (7, 3), (2, 4)])
def test_mask_brute_force_sets(n, K):
    anchor, depth = inputs.full_grid(n, K)
    rng = np.random.default_rng(n * 10 + K)
    perm = rng.permutation(n * K)            # the mask depends on metadata only, not on order
    anchor, depth = anchor[perm], depth[perm]
    assert np.array_equal(orc.mask_dense(anchor, depth), dense_from_sets(anchor, depth))


def test_mask_never_sees_later_depth_or_other_chain():
    anchor, depth = inputs.full_grid(6, 4)
    M = orc.mask_dense(anchor, depth)
    for q in range(24):
        for k in range(24):
            if M[q, k]:
                assert depth[k] <= depth[q]
                assert depth[k] == 0 or anchor[k] == anchor[q]
                assert anchor[k] + depth[k] <= anchor[q] + depth[q]   # never a later position
        assert M[q, q] == 1


def test_mask_sequences_do_not_mix():
    a1, d1 = inputs.full_grid(3, 2)
    anchor, depth = np.concatenate([a1, a1]), np.concatenate([d1, d1])
    seq = np.repeat(np.arange(2, dtype=np.int32), 6)
    M = orc.mask_dense(anchor, depth, seq)
    assert M[:6, 6:].sum() == 0 and M[6:, :6].sum() == 0
    assert np.array_equal(M[:6, :6], M[6:, 6:])
    assert np.array_equal(M[:6, :6], orc.mask_dense(a1, d1))


@pytest.mark.parametrize("n,K", [(128, 4), (512, 8), (1024, 8)])
def test_pair_count_closed_form(n, K):
    anchor, depth = inputs.full_grid(n, K)
    want = K * n * (n + 1) // 2 + n * K * (K - 1) // 2   # causal triangle per depth + chains
    assert orc.count_pairs(anchor, depth) == want


def test_position_invariance_top_left_submatrix():
    """Section 3.1 / Figure 2: the mask of a shorter sequence is the top-left block of a longer
    one's (tokens interleaved anchor-major so that a prefix of tokens is a prefix of anchors)."""
    K = 4

    def interleaved(n):
        anchor = np.repeat(np.arange(n, dtype=np.int32), K)
        depth = np.tile(np.arange(K, dtype=np.int32), n)
        return anchor, depth

    big = orc.mask_dense(*interleaved(12))
    for n in (1, 5, 9):
        small = orc.mask_dense(*interleaved(n))
        assert np.array_equal(small, big[: n * K, : n * K])


def test_fig3_example_counts_and_pairs():
    P, total = read_fig3()
    assert sum(len(p) for p in P) == total == 38
    for g in range(1, 4):                      # chains are nested: p at depth g has p-1 at g-1
        assert all((p - 1) in P[g - 1] for p in P[g])
    _, anchor, depth = fig3_tokens()
    # a token at position p sees p+1 keys (anchor+1 real tokens and `depth` chain tokens)
    want = sum(p + 1 for ps in P for p in ps)
    assert want == 344
    assert orc.count_pairs(anchor, depth) == want
    assert np.array_equal(orc.mask_dense(anchor, depth), dense_from_sets(anchor, depth))


def test_cod_position_count():
    assert round(opart.cod_total_positions(8192, 8, 0.8)) == 34088     # "approximately 34K"
    assert opart.cod_total_positions(16, 4, 1.0 - 1e-12) == pytest.approx(64, rel=1e-9)


# ---------------------------------------------------------------- Algorithm 1
def test_alg1_fig3_dependencies_colocated():
    P, _ = read_fig3()
    A, N, B = opart.assign_segments(P, S=2, L=16)
    assert B == [0, 8, 16]
    assert A[2][8] == A[1][7] == 0             # the violation the paper names is avoided
    for g in range(2, 4):
        for p in P[g]:
            assert A[g][p] == A[g - 1][p - 1]
    for g in (0, 1):
        for p in P[g]:
            assert A[g][p] == (0 if p < 8 else 1)
    assert N[0] == list(range(8)) and N[1] == list(range(16))
    sizes = [[sum(1 for p in P[g] if A[g][p] == s) for g in range(4)] for s in range(2)]
    # by hand: depth1 {1,3,4,6,7 | 9,10,12,14,15}; depth2 {2,5,7,8 | 11,13,15}; depth3 {3,6,9 | 12,14}
    assert sizes == [[8, 5, 4, 3], [8, 5, 3, 2]]


@pytest.mark.parametrize("n,K,S", [(16, 4, 2), (37, 5, 4), (64, 8, 3)])
def test_alg1_key_sets_are_dependency_closed(n, K, S):
    anchor, depth = inputs.full_grid(n, K)
    P = inputs.position_sets(anchor, depth, K)
    A, N, B = opart.assign_segments(P, S, n)
    seg = np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)
    for a, d, s in zip(anchor, depth, seg):
        for (ak, dk) in chain_set(int(a), int(d)):
            if dk == 0:
                assert ak in N[s]               # cumulative depth-0 context covers it
            else:
                assert A[dk][ak + dk] == s      # chain tokens share the segment


# ---------------------------------------------------------------- tile classes
def test_tile_class_counts_closed_form():
    n, K, B = 1024, 4, 128
    anchor, depth = inputs.full_grid(n, K)
    cls, ks, kl = orc.classify_tiles(anchor, depth, 0, n * K, None, B, B)
    t = n // B
    assert cls.shape == (K * t, K * t)
    assert int((cls == 2).sum()) == K * t * (t - 1) // 2
    assert int((cls == 1).sum()) == K * t + t * K * (K - 1) // 2
    assert np.array_equal(ks, np.arange(K * t) * B) and np.all(kl == B)


def test_tile_classes_from_dense_mask_ragged():
    n, K, BM, BN = 37, 3, 16, 8
    anchor, depth = inputs.full_grid(n, K)
    M = orc.mask_dense(anchor, depth)
    q0, q1, kr = 5, 90, [(0, 37), (40, 111)]
    cls, ks, kl = orc.classify_tiles(anchor, depth, q0, q1, kr, BM, BN)
    tiles = [(b, min(b + BN, e)) for (s, e) in kr for b in range(s, e, BN)]
    assert [t[0] for t in tiles] == ks.tolist() and [t[1] - t[0] for t in tiles] == kl.tolist()
    for qt in range(cls.shape[0]):
        r0, r1 = q0 + qt * BM, min(q0 + qt * BM + BM, q1)
        for kt, (b, e) in enumerate(tiles):
            sub = M[r0:r1, b:e]
            want = 0 if sub.sum() == 0 else (2 if (e - b == BN and sub.all()) else 1)
            assert cls[qt, kt] == want


# ---------------------------------------------------------------- forward
def test_depth0_rows_are_causal_attention():
    n, K, Hq, Hkv, D = 48, 4, 4, 2, 16
    anchor, depth, Q, Kt, V, _ = rand_case(n, K, Hq, Hkv, D, seed=3, std=1.0)
    scale = 1 / math.sqrt(D)
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, scale, rows=np.arange(n))
    q = Q[:n].double().permute(1, 0, 2)[None]
    k = Kt[:n].double().repeat_interleave(Hq // Hkv, 1).permute(1, 0, 2)[None]
    v = V[:n].double().repeat_interleave(Hq // Hkv, 1).permute(1, 0, 2)[None]
    ref = F.scaled_dot_product_attention(q, k, v, is_causal=True, scale=scale)[0].permute(1, 0, 2)
    assert np.allclose(O, ref.numpy(), rtol=0, atol=1e-12)


def test_k1_is_plain_causal_attention_fwd_bwd():
    n, Hq, Hkv, D = 40, 4, 2, 8
    anchor, depth, Q, Kt, V, dO = rand_case(n, 1, Hq, Hkv, D, seed=4, std=1.0)
    scale = 0.37
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, scale)
    dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, scale)
    q = Q.double().requires_grad_()
    k = Kt.double().requires_grad_()
    v = V.double().requires_grad_()
    kx = k.repeat_interleave(Hq // Hkv, 1)
    vx = v.repeat_interleave(Hq // Hkv, 1)
    ref = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None], kx.permute(1, 0, 2)[None],
                                         vx.permute(1, 0, 2)[None], is_causal=True, scale=scale)
    ref = ref[0].permute(1, 0, 2)
    (ref * dO.double()).sum().backward()
    assert np.allclose(O, ref.detach().numpy(), atol=1e-12)
    assert np.allclose(dQ, q.grad.numpy(), atol=1e-11)
    assert np.allclose(dK, k.grad.numpy(), atol=1e-11)
    assert np.allclose(dV, v.grad.numpy(), atol=1e-11)


def test_last_chain_equals_inference_layout():
    """Rows (n-1, 0..K-1) see [all real tokens, own chain]: plain causal attention over that
    concatenation, which is the drafter's single-pass inference layout (Section 2)."""
    n, K, Hq, Hkv, D = 20, 5, 2, 1, 16
    anchor, depth, Q, Kt, V, _ = rand_case(n, K, Hq, Hkv, D, seed=5, std=1.0)
    rows = np.array([d * n + (n - 1) for d in range(K)])
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, 0.25, rows=rows)
    idx = torch.tensor(list(range(n)) + [d * n + (n - 1) for d in range(1, K)])
    q = Q[idx].double().permute(1, 0, 2)[None]
    k = Kt[idx].double().repeat_interleave(Hq, 1).permute(1, 0, 2)[None]
    v = V[idx].double().repeat_interleave(Hq, 1).permute(1, 0, 2)[None]
    ref = F.scaled_dot_product_attention(q, k, v, is_causal=True, scale=0.25)[0].permute(1, 0, 2)
    assert np.allclose(O, ref[n - 1:].numpy(), atol=1e-12)


def test_rows_are_softmax_over_exactly_the_allowed_set():
    n, K = 6, 3
    T = n * K
    anchor, depth = inputs.full_grid(n, K)
    g = torch.Generator().manual_seed(7)
    Q = torch.randn(T, 1, 4, generator=g)
    Kt = torch.randn(T, 1, 4, generator=g)
    V = torch.eye(T)[:, None, :]                   # O row = the probabilities themselves
    Qp = torch.zeros(T, 1, T); Qp[..., :4] = Q
    Kp = torch.zeros(T, 1, T); Kp[..., :4] = Kt
    O, LSE = orc.attn_fwd(anchor, depth, Qp, Kp, V, 1.0)
    M = dense_from_sets(anchor, depth)
    P = O[:, 0, :]
    assert np.allclose(P.sum(1), 1.0, atol=1e-14)
    assert np.all(P[M == 0] == 0.0) and np.all(P[M == 1] > 0.0)
    S = (Q[:, 0].double() @ Kt[:, 0].double().T).numpy()
    for q in range(T):
        s = S[q][M[q] == 1]
        assert LSE[q, 0] == pytest.approx(np.log(np.exp(s).sum()), rel=1e-13)
        assert np.allclose(P[q][M[q] == 1], np.exp(s) / np.exp(s).sum(), atol=1e-14)


def test_forward_matches_dense_mask_torch_with_gqa_and_shuffle():
    n, K, Hq, Hkv, D = 11, 4, 6, 2, 8
    anchor, depth, Q, Kt, V, _ = rand_case(n, K, Hq, Hkv, D, seed=8, std=1.0)
    perm = np.random.default_rng(1).permutation(n * K)
    anchor, depth = anchor[perm], depth[perm]
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, 0.3)
    ref_O, ref_L = torch_dense_attention(dense_from_sets(anchor, depth), Q.double(), Kt.double(),
                                         V.double(), 0.3)
    assert np.allclose(O, ref_O.numpy(), atol=1e-12)
    assert np.allclose(LSE, ref_L.numpy(), atol=1e-12)


def test_empty_row_gives_zero_and_minus_inf():
    anchor, depth = inputs.full_grid(4, 2)
    _, _, Q, Kt, V, dO = rand_case(4, 2, 2, 1, 8, seed=9)
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, 1.0, rows=[0, 5], kranges=[(2, 4)])
    assert np.all(O == 0) and np.all(np.isneginf(LSE))       # neither row sees tokens 2..3
    dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, 1.0, rows=[0, 5], kranges=[(2, 4)])
    assert np.all(dQ == 0) and np.all(dK == 0) and np.all(dV == 0)


# ---------------------------------------------------------------- backward
def test_backward_matches_autograd_of_dense_formulation():
    n, K, Hq, Hkv, D = 9, 4, 4, 2, 8
    anchor, depth, Q, Kt, V, dO = rand_case(n, K, Hq, Hkv, D, seed=10, std=1.0)
    q = Q.double().requires_grad_()
    k = Kt.double().requires_grad_()
    v = V.double().requires_grad_()
    O, _ = torch_dense_attention(dense_from_sets(anchor, depth), q, k, v, 0.41)
    (O * dO.double()).sum().backward()
    dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, 0.41)
    assert np.allclose(dQ, q.grad.numpy(), atol=1e-11)
    assert np.allclose(dK, k.grad.numpy(), atol=1e-11)
    assert np.allclose(dV, v.grad.numpy(), atol=1e-11)


def test_backward_central_finite_differences():
    n, K, Hq, Hkv, D = 5, 3, 2, 1, 4
    anchor, depth, Q, Kt, V, dO = rand_case(n, K, Hq, Hkv, D, seed=11, std=1.0)
    scale = 0.5
    dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, scale)
    eps = 2.0 ** -10                       # exactly representable on top of bf16 values in fp32
    base = [Q.float().numpy(), Kt.float().numpy(), V.float().numpy()]
    dOd = dO.double().numpy()

    def loss(arrs):
        O, _ = orc.attn_fwd(anchor, depth, arrs[0], arrs[1], arrs[2], scale)
        return float((O * dOd).sum())

    rng = np.random.default_rng(0)
    for which, grad in enumerate((dQ, dK, dV)):
        flat = grad.reshape(-1)
        for idx in rng.choice(flat.size, size=25, replace=False):
            arrs = [a.copy() for a in base]
            arrs[which].reshape(-1)[idx] += eps
            up = loss(arrs)
            arrs[which].reshape(-1)[idx] -= 2 * eps
            dn = loss(arrs)
            fd = (up - dn) / (2 * eps)
            assert fd == pytest.approx(flat[idx], rel=2e-5, abs=1e-7)


# ---------------------------------------------------------------- partitioning
@pytest.mark.parametrize("case", ["full_grid", "fig3"])
def test_partitioned_equals_unpartitioned(case):
    if case == "full_grid":
        n, K, S = 29, 4, 3
        anchor, depth = inputs.full_grid(n, K)
        P = inputs.position_sets(anchor, depth, K)
    else:
        n, K, S = 16, 4, 2
        P, anchor, depth = fig3_tokens()
    A, N, B = opart.assign_segments(P, S, n)
    seg = np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)
    perm = inputs.arrange_by_segment(anchor, depth, seg)
    anchor, depth, seg = anchor[perm], depth[perm], seg[perm]
    T = len(anchor)
    Q, Kt, V, dO = inputs.make_tensors(T, 4, 2, 8, seed=12, q_std=1.0)
    O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, 0.35)
    dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, 0.35)
    parts = inputs.partitions_from_layout(seg, depth)
    assert len(parts) == S and sum(p["q"][1] - p["q"][0] for p in parts) == T
    dKp = np.zeros_like(dK)
    dVp = np.zeros_like(dV)
    for p in parts:
        rows = np.arange(*p["q"])
        Op, Lp = orc.attn_fwd(anchor, depth, Q, Kt, V, 0.35, rows=rows, kranges=p["k"])
        dQp, _, _ = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, 0.35, rows=rows, kranges=p["k"],
                                 dK=dKp, dV=dVp)
        assert np.allclose(Op, O[rows], atol=1e-13) and np.allclose(Lp, LSE[rows], atol=1e-13)
        assert np.allclose(dQp, dQ[rows], atol=1e-12)
        # the visible key set of a partition covers every allowed key of its queries
        vis = np.zeros(T, bool)
        for (b, e) in p["k"]:
            vis[b:e] = True
        M = orc.mask_dense(anchor, depth)
        assert not M[rows][:, ~vis].any()
    assert np.allclose(dKp, dK, atol=1e-12) and np.allclose(dVp, dV, atol=1e-12)


# ---------------------------------------------------------------- visible key ranges
def hidden_mask(anchor, depth, kranges):
    """The mask with the columns outside the half-open ranges zeroed by hand."""
    M = dense_from_sets(anchor, depth).copy()
    vis = np.zeros(len(anchor), bool)
    for b, e in kranges:
        vis[b:e] = True
    M[:, ~vis] = 0
    return M


def test_key_ranges_hide_part_of_the_allowed_set():
    """A partition's visible ranges cut into rows' allowed sets: ranges that end one token before
    and one token after an allowed key, a gap in the middle, and a range starting past token 0.
    Forward, backward and the pair count must equal the dense formulation on a mask whose hidden
    columns this test zeroes itself (half-open ranges: `begin` is visible, `end` is not)."""
    n, K, Hq, Hkv, D = 10, 4, 4, 2, 8
    anchor, depth, Q, Kt, V, dO = rand_case(n, K, Hq, Hkv, D, seed=21, std=1.0)
    perm = np.random.default_rng(5).permutation(n * K)
    anchor, depth = anchor[perm], depth[perm]
    T = n * K
    full = dense_from_sets(anchor, depth)
    # pick a row with many allowed keys and cut right before / right after two of them
    q_big = int(np.argmax(full.sum(1)))
    ks = np.nonzero(full[q_big])[0]
    k_lo, k_hi = int(ks[1]), int(ks[-2])
    assert k_lo + 1 < k_hi
    cases = [
        [(0, k_lo), (k_lo + 1, k_hi + 1)],      # ends one before an allowed key; k_hi is the last visible
        [(1, k_lo + 1), (k_hi, T)],             # ends one after it (k_lo visible); token 0 hidden
        [(3, 17), (18, 19), (25, T - 2)],       # three ranges, one of a single token
    ]
    for kr in cases:
        M = hidden_mask(anchor, depth, kr)
        part = M.sum(1)
        assert ((part > 0) & (part < full.sum(1))).sum() >= 5      # rows hidden only in part
        assert orc.count_pairs(anchor, depth, kranges=kr) == int(M.sum())
        rows = np.arange(T)
        assert orc.count_pairs(anchor, depth, rows=rows[::3], kranges=kr) == int(M[::3].sum())
        q = Q.double().requires_grad_()
        k = Kt.double().requires_grad_()
        v = V.double().requires_grad_()
        live = torch.as_tensor(M.sum(1) > 0)
        ref_O, ref_L = torch_dense_attention(M[live.numpy()], q[live], k, v, 0.29)
        (ref_O * dO.double()[live]).sum().backward()
        O, LSE = orc.attn_fwd(anchor, depth, Q, Kt, V, 0.29, kranges=kr)
        dQ, dK, dV = orc.attn_bwd(anchor, depth, Q, Kt, V, dO, 0.29, kranges=kr)
        lv = live.numpy()
        assert np.allclose(O[lv], ref_O.detach().numpy(), atol=1e-12)
        assert np.allclose(LSE[lv], ref_L.detach().numpy(), atol=1e-12)
        assert np.all(O[~lv] == 0) and np.all(np.isneginf(LSE[~lv]))
        assert np.allclose(dQ, q.grad.numpy(), atol=1e-11)       # rows that see nothing: zero
        assert np.allclose(dK, k.grad.numpy(), atol=1e-11)
        assert np.allclose(dV, v.grad.numpy(), atol=1e-11)
        hidden = np.ones(T, bool)
        for b, e in kr:
            hidden[b:e] = False
        assert np.all(dK[hidden] == 0) and np.all(dV[hidden] == 0)


@pytest.mark.parametrize("case", ["full_grid", "fig3", "cod"])
def test_layout_key_ranges_are_alg1_cumulative_depth0_sets(case):
    """Algorithm 1, phase 3: segment s sees the depth-0 positions p < B[s+1].  The ranges the
    layout helper hands to both sides must hold, outside the segment's own block, exactly the
    depth-0 tokens of N[s] that earlier segments own -- token for token."""
    if case == "full_grid":
        n, K, S = 45, 5, 4
        anchor, depth = inputs.full_grid(n, K)
    elif case == "fig3":
        n, K, S = 16, 4, 2
        _, anchor, depth = fig3_tokens()
    else:
        n, K, S = 60, 6, 3
        anchor, depth = inputs.cod_grid(n, K, 0.7, seed=2)
    P = inputs.position_sets(anchor, depth, K)
    A, N, B = opart.assign_segments(P, S, n)
    seg = np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)
    perm = inputs.arrange_by_segment(anchor, depth, seg)
    anchor, depth, seg = anchor[perm], depth[perm], seg[perm]
    parts = inputs.partitions_from_layout(seg, depth)
    assert len(parts) == S
    for s, p in enumerate(parts):
        own = set(range(*p["q"]))
        assert own == set(np.nonzero(seg == s)[0].tolist())
        vis = set()
        for b, e in p["k"]:
            vis |= set(range(b, e))
        assert own <= vis
        outside = vis - own
        assert all(depth[t] == 0 for t in outside)
        # depth-0 positions visible to segment s, as Algorithm 1 lists them
        vis_d0 = sorted(int(anchor[t]) for t in vis if depth[t] == 0)
        assert vis_d0 == N[s]
