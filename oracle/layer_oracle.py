"""TEST INFRASTRUCTURE: fp64 CPU oracle of the attention half of a drafter layer run segment by
segment, as Section 3.2 and Algorithm 1 describe training on long sequences.

Only the tests, the smoke check and the benchmark's CPU legs may import this module; it never
touches the CUDA library.

What it computes.  The drafter is a LLaMA-3-style layer (Section 2).  For hidden rows X [T, d_model]
of the expanded sequence and the fused projection weight W [(Hq + 2 Hkv) D, d_model]:

    qkv = X W^T                         one fused row per token: query | key | value heads
    Q, K, V = rotary(qkv)               positions p = anchor + depth (rope_oracle)
    O, LSE  = masked attention(Q, K, V) the parallel-prediction mask (peagle_oracle's predicate)
    loss    = <O, dO>                   dO stands for the gradient that reaches O

and the gradients dX, dW of that loss.  Run on the whole sequence this is `layer_whole`.  Run as
the paper trains (Section 3.2, "Our solution"; Algorithm 1 phase 3) every segment s is a separate
forward-backward pass over its own tokens plus the depth-0 tokens of earlier segments, whose K / V
are projected AGAIN inside segment s (they are keys only: each token is a query in exactly one
segment), and the gradients of the segments are added (within-sequence gradient accumulation):
`layer_segmented`.  Both must agree to rounding: that identity is one of the pins.

The attention inside is written here a second time, in numpy on fp64 arrays with the mask
materialised per block of rows (the C oracle takes fp32 arrays of bf16 values, which would round
the projected Q / K / V).  It is pinned to the C oracle on bf16 inputs.
"""
from __future__ import annotations

import numpy as np

from oracle import rope_oracle as ro


def allowed_matrix(anchor_q, depth_q, anchor_k, depth_k) -> np.ndarray:
    """Section 3 / 3.2: query (a_q, d_q) sees key (a_k, d_k) iff the key is a real context token
    not after the query's anchor, or a token of the query's own chain at the same or an earlier
    depth.  Boolean [nq, nk]."""
    aq, dq = np.asarray(anchor_q)[:, None], np.asarray(depth_q)[:, None]
    ak, dk = np.asarray(anchor_k)[None, :], np.asarray(depth_k)[None, :]
    return ((dk == 0) & (ak <= aq)) | ((dk > 0) & (ak == aq) & (dk <= dq))


def attention_np(anchor, depth, Q, K, V, dO, scale, rows, block: int = 256):
    """Masked softmax attention and its gradients in fp64 for query rows `rows` (indices into the
    given token arrays) over all given tokens as keys.  Q [T, Hq, D], K, V [T, Hkv, D], dO
    [len(rows), Hq, D].  Returns O, LSE [len(rows), Hq(, D)], dQ [len(rows), Hq, D], dK, dV [T, Hkv, D]."""
    Q, K, V, dO = (np.asarray(t, np.float64) for t in (Q, K, V, dO))
    anchor, depth, rows = np.asarray(anchor), np.asarray(depth), np.asarray(rows)
    T, Hq, D = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    n = rows.shape[0]
    O = np.zeros((n, Hq, D))
    LSE = np.full((n, Hq), -np.inf)
    dQ = np.zeros((n, Hq, D))
    dK = np.zeros((T, Hkv, D))
    dV = np.zeros((T, Hkv, D))
    for b in range(0, n, block):
        r = rows[b:b + block]
        M = allowed_matrix(anchor[r], depth[r], anchor, depth)          # [nb, T]
        for h in range(Hq):
            g = h // G
            S = scale * (Q[r, h] @ K[:, g].T)
            S = np.where(M, S, -np.inf)
            m = S.max(axis=1, keepdims=True)
            live = np.isfinite(m[:, 0])
            m = np.where(np.isfinite(m), m, 0.0)
            E = np.exp(S - m)
            l = E.sum(axis=1, keepdims=True)
            P = np.where(l > 0, E / np.where(l > 0, l, 1.0), 0.0)
            O[b:b + block, h] = P @ V[:, g]
            LSE[b:b + block, h] = np.where(live, m[:, 0] + np.log(np.where(l[:, 0] > 0, l[:, 0], 1.0)), -np.inf)
            g_o = dO[b:b + block, h]
            dP = g_o @ V[:, g].T
            delta = (g_o * O[b:b + block, h]).sum(axis=1, keepdims=True)
            dS = P * (dP - delta)
            dQ[b:b + block, h] = scale * (dS @ K[:, g])
            dK[:, g] += scale * (dS.T @ Q[r, h])
            dV[:, g] += P.T @ g_o
    return O, LSE, dQ, dK, dV


def _pass(X, W, anchor, depth, Hq, Hkv, D, base, scale, dO_rows, rows, vis):
    """One forward-backward pass of the chain on the tokens `vis` (indices, ascending) with the
    queries `rows` (a subset of vis).  Returns O, LSE of the rows and the pass's dX [len(vis),
    d_model], dW."""
    Xv = X[vis]
    qkv = Xv @ W.T                                                   # projection of every visible token
    Q, K, V = ro.rope_qkv_fwd(qkv, anchor[vis], depth[vis], Hq, Hkv, D, base)
    local = np.searchsorted(vis, rows)
    assert np.array_equal(vis[local], rows)
    O, LSE, dQ_r, dK, dV = attention_np(anchor[vis], depth[vis], Q, K, V, dO_rows, scale, local)
    dQ = np.zeros_like(Q)
    dQ[local] = dQ_r                                                # tokens that are keys only get no dQ
    d_qkv = ro.rope_qkv_bwd(dQ, dK, dV, anchor[vis], depth[vis], Hq, Hkv, D, base)
    return O, LSE, d_qkv @ W, d_qkv.T @ Xv


def layer_whole(X, W, anchor, depth, Hq, Hkv, D, base, scale, dO):
    """The chain on the whole sequence in one pass.  Returns O [T, Hq, D], LSE [T, Hq], dX, dW."""
    X, W, dO = (np.asarray(t, np.float64) for t in (X, W, dO))
    anchor, depth = np.asarray(anchor), np.asarray(depth)
    T = X.shape[0]
    every = np.arange(T)
    return _pass(X, W, anchor, depth, Hq, Hkv, D, base, scale, dO, every, every)


def layer_segmented(X, W, anchor, depth, Hq, Hkv, D, base, scale, dO, parts):
    """The chain as Section 3.2 trains it: one forward-backward pass per segment over the
    segment's tokens and the keys it may see (`parts`: dicts {q: (b, e), k: [(b, e), ...]}, the
    ranges Algorithm 1's phase 3 yields), K / V of earlier depth-0 tokens projected again in
    every segment that sees them, dX and dW summed over the segments."""
    X, W, dO = (np.asarray(t, np.float64) for t in (X, W, dO))
    anchor, depth = np.asarray(anchor), np.asarray(depth)
    T = X.shape[0]
    O = np.zeros((T, Hq, D))
    LSE = np.zeros((T, Hq))
    dX = np.zeros_like(X)
    dW = np.zeros_like(W)
    for p in parts:
        rows = np.arange(*p["q"])
        vis = np.concatenate([np.arange(b, e) for b, e in p["k"]])
        O[rows], LSE[rows], dX_s, dW_s = _pass(X, W, anchor, depth, Hq, Hkv, D, base, scale,
                                               dO[rows], rows, vis)
        dX[vis] += dX_s                                              # gradient accumulation
        dW += dW_s
    return O, LSE, dX, dW
