"""TEST INFRASTRUCTURE: fp64 CPU oracle of the drafter layer's rotary prologue.

Only the tests and the smoke check may import this module; it never touches the CUDA library.

What it computes (Section 2: the drafter is a LLaMA-3-style layer with rotary position
embeddings, RoFormer's construction; Appendix B works with the rotation R_p of a token at
sequence position p).  A token of the expanded sequence with anchor a and depth d stands at
sequence position p = a + d (depth k predicts the token k + 1 positions ahead of the context
token it hangs from; Section 3).  The prologue takes the fused projection output of the layer,
one row per token holding [Hq query heads | Hkv key heads | Hkv value heads] of D elements each,
and produces the three tensors the attention reads: Q [T, Hq, D] and K [T, Hkv, D] rotated by R_p,
V [T, Hkv, D] copied.  R_p acts on a head vector x pair by pair, LLaMA's half-split pairing
(element i with element i + D/2, i < D/2):

    angle_i = p * base ** (-2 i / D)
    y[i]       = x[i] * cos(angle_i) - x[i + D/2] * sin(angle_i)
    y[i + D/2] = x[i + D/2] * cos(angle_i) + x[i] * sin(angle_i)

The backward pass is the transpose: the gradient of a rotated vector is rotated by R_{-p}.
Everything is written out from that definition in float64, no blocking or fusion.
"""
from __future__ import annotations

import numpy as np


def rope_angles(pos, D: int, base: float) -> np.ndarray:
    """angle[t, i] = pos[t] * base ** (-2 i / D) for i < D / 2 (float64)."""
    pos = np.asarray(pos, dtype=np.float64)
    i = np.arange(D // 2, dtype=np.float64)
    inv_freq = np.power(np.float64(base), -2.0 * i / np.float64(D))
    return pos[:, None] * inv_freq[None, :]


def rotate(x: np.ndarray, angle: np.ndarray) -> np.ndarray:
    """R applied to x [T, H, D] with angle [T, D/2]; half-split pairing."""
    x = np.asarray(x, dtype=np.float64)
    half = x.shape[-1] // 2
    c = np.cos(angle)[:, None, :]
    s = np.sin(angle)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def rope_qkv_fwd(qkv, anchor, depth, Hq: int, Hkv: int, D: int, base: float):
    """qkv [T, (Hq + 2 Hkv) * D] -> (Q [T, Hq, D], K [T, Hkv, D], V [T, Hkv, D]), float64."""
    qkv = np.asarray(qkv, dtype=np.float64)
    T = qkv.shape[0]
    pos = np.asarray(anchor, dtype=np.int64) + np.asarray(depth, dtype=np.int64)
    angle = rope_angles(pos, D, base)
    q = qkv[:, : Hq * D].reshape(T, Hq, D)
    k = qkv[:, Hq * D : (Hq + Hkv) * D].reshape(T, Hkv, D)
    v = qkv[:, (Hq + Hkv) * D :].reshape(T, Hkv, D)
    return rotate(q, angle), rotate(k, angle), v.copy()


def rope_qkv_bwd(dQ, dK, dV, anchor, depth, Hq: int, Hkv: int, D: int, base: float):
    """Gradient with respect to the fused row: [T, (Hq + 2 Hkv) * D], float64."""
    dQ = np.asarray(dQ, dtype=np.float64)
    dK = np.asarray(dK, dtype=np.float64)
    dV = np.asarray(dV, dtype=np.float64)
    T = dQ.shape[0]
    pos = np.asarray(anchor, dtype=np.int64) + np.asarray(depth, dtype=np.int64)
    angle = rope_angles(pos, D, base)
    gq = rotate(dQ, -angle).reshape(T, Hq * D)
    gk = rotate(dK, -angle).reshape(T, Hkv * D)
    return np.concatenate([gq, gk, dV.reshape(T, Hkv * D)], axis=1)
