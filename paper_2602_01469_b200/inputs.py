"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests/benchmark.

This module holds no arithmetic of the method: it draws random tensors, lays tokens out in
memory and lists the benchmark workloads.  It imports neither the oracle nor the CUDA binding.

The workloads stand in for the paper's long reasoning traces (Figure 1: median 3,891 tokens,
P90 10,800, P99 about 20,000) with K = 8 depths and 8,192-token segments (Section 5.1).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    seq_lens: tuple          # context tokens n per sequence
    K: int                   # prediction depths
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_segments: int = 1      # segments per sequence (even boundaries), when seg_len is None
    seg_len: int | None = None   # fixed segment length in context tokens (overrides n_segments)
    seed: int = 0
    cod_r: float | None = None   # COD retention rate (Section 3): depth d keeps about n * r^d chains
    # memory order inside a segment: "depth_major" = G0 | G1 | ... blocks (Figures 2-3);
    # "anchor_major" = the depth-0 block, then the deeper tokens chain by chain (anchor, depth)
    order: str = "depth_major"

    @property
    def total_tokens(self) -> int:
        if self.cod_r is not None:
            return sum(int(cod_grid(n, self.K, self.cod_r, self.seed + i)[0].shape[0])
                       for i, n in enumerate(self.seq_lens))
        return sum(self.seq_lens) * self.K

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


def longtail_lengths(total: int = 65536, seed: int = 0) -> tuple:
    """Sequence lengths for the long-tail batch: lognormal with median 3,891 and P90 10,800
    (Figure 1), rounded, clipped to [1, 20480], drawn until ``total`` context tokens are
    reached (the last one truncated)."""
    mu = math.log(3891.0)
    sigma = math.log(10800.0 / 3891.0) / 1.2815515655446004
    rng = np.random.default_rng(seed)
    out, acc = [], 0
    while acc < total:
        n = int(min(max(round(float(rng.lognormal(mu, sigma))), 1), 20480))
        n = min(n, total - acc)
        out.append(n)
        acc += n
    return tuple(out)


WORKLOADS = {
    "tiny": Workload("tiny", (128,), 4, 4, 1, 64, seed=0),
    "qwen3coder_n2048": Workload("qwen3coder_n2048", (2048,), 8, 32, 4, 128, seed=20),
    "gptoss_n4096": Workload("gptoss_n4096", (4096,), 8, 64, 8, 64, seed=30),
    "p90_n11008_s4": Workload("p90_n11008_s4", (11008,), 8, 64, 8, 64, n_segments=4, seed=40),
    "longtail_varlen": Workload("longtail_varlen", longtail_lengths(), 8, 64, 8, 64,
                                seg_len=8192, seed=50),
}
# a half-length copy of the headline shape, small enough for profiler captures
# the paper's own example of Section 3.2: 8,192 tokens, K = 8, retention 0.8 (about 34K positions)
WORKLOADS["gptoss_n8192_cod"] = Workload("gptoss_n8192_cod", (8192,), 8, 64, 8, 64, seed=60, cod_r=0.8)
WORKLOADS["gptoss_n2048_profile"] = Workload("gptoss_n2048_profile", (2048,), 8, 64, 8, 64, seed=31)
# the headline grid with a chain's tokens stored next to each other: a second workload, not the headline
WORKLOADS["gptoss_n4096_anchor_major"] = Workload("gptoss_n4096_anchor_major", (4096,), 8, 64, 8, 64,
                                                  seed=30, order="anchor_major")
HEADLINE = "gptoss_n4096"


def full_grid(n: int, K: int):
    """All n anchors at every one of the K depths, depth-major (G0 | G1 | ... blocks)."""
    depth = np.repeat(np.arange(K, dtype=np.int32), n)
    anchor = np.tile(np.arange(n, dtype=np.int32), K)
    return anchor, depth


def cod_grid(n: int, K: int, r: float, seed: int):
    """COD down-sampling of the full grid (Section 3: depth 0 keeps all n positions, depth d
    about n * r^d, drawn at random per example; Section 3.2: position p at depth d needs position
    p-1 at depth d-1, so the sets are nested along chains).  Depth d keeps round(r * kept(d-1)) of
    the chains still alive at depth d-1, chosen uniformly with ``numpy.random.default_rng(seed)``;
    a chain whose position anchor + d would pass the end of the sequence is not continued, as in
    the printed example.  Returns anchor, depth (depth-major, anchors ascending)."""
    rng = np.random.default_rng(seed)
    alive = np.arange(n, dtype=np.int32)
    anchors, depths = [alive], [np.zeros(n, np.int32)]
    for d in range(1, K):
        alive = alive[alive + d < n]
        keep = min(int(round(r * anchors[-1].shape[0])), alive.shape[0])
        alive = np.sort(rng.choice(alive, size=keep, replace=False)).astype(np.int32)
        anchors.append(alive)
        depths.append(np.full(keep, d, np.int32))
    return np.concatenate(anchors), np.concatenate(depths)


def position_sets(anchor: np.ndarray, depth: np.ndarray, K: int) -> list:
    """Algorithm 1's input P: the sequence positions p = anchor + depth kept at each depth."""
    return [sorted((anchor[depth == g] + g).tolist()) for g in range(K)]


def segment_boundaries(n: int, n_segments: int = 1, seg_len: int | None = None) -> list:
    """Boundaries in context-token space: even split, or fixed-length segments."""
    if seg_len is not None:
        b = list(range(0, n, seg_len)) + [n]
        return b
    return [(k * n) // n_segments for k in range(n_segments + 1)]


def arrange_by_segment(anchor: np.ndarray, depth: np.ndarray, segment: np.ndarray,
                       order: str = "depth_major"):
    """Memory order of one sequence: segments contiguous; inside a segment either depth-major
    (anchors ascending inside a depth) or the depth-0 block followed by the deeper tokens
    anchor-major, so that a chain's tokens are neighbours.  Returns the permutation."""
    if order == "anchor_major":
        return np.lexsort((depth, anchor, depth > 0, segment))
    assert order == "depth_major"
    return np.lexsort((anchor, depth, segment))


def partitions_from_layout(segment: np.ndarray, depth: np.ndarray, offset: int = 0) -> list:
    """Query range and visible key ranges of every segment of one sequence laid out by
    ``arrange_by_segment``: a segment's queries are its own block; its keys are the depth-0
    sub-blocks of all earlier segments plus its whole block.  Ranges are half-open token
    indices shifted by ``offset`` (the sequence's first token in the batch)."""
    S = int(segment.max()) + 1 if segment.size else 0
    parts = []
    d0_blocks = []
    for s in range(S):
        idx = np.nonzero(segment == s)[0]
        if idx.size == 0:
            continue
        b, e = int(idx[0]), int(idx[-1]) + 1
        assert np.all(segment[b:e] == s), "segments must be contiguous"
        keys = list(d0_blocks) + [(b + offset, e + offset)]
        merged = []
        for r in keys:                       # merge touching ranges
            if merged and merged[-1][1] == r[0]:
                merged[-1] = (merged[-1][0], r[1])
            else:
                merged.append(r)
        parts.append({"q": (b + offset, e + offset), "k": merged})
        n0 = int(np.count_nonzero(depth[b:e] == 0))
        assert np.all(depth[b:b + n0] == 0)
        if n0:
            d0_blocks.append((b + offset, b + n0 + offset))
    return parts


def make_tensors(T: int, Hq: int, Hkv: int, D: int, seed: int, q_std: float | None = None):
    """bf16 Q, K, V ~ N(0,1)/sqrt(D) (or N(0, q_std^2)) and dO ~ N(0,1), CPU tensors."""
    std = 1.0 / math.sqrt(D) if q_std is None else q_std
    out = []
    for i, (H, s) in enumerate(((Hq, std), (Hkv, std), (Hkv, std), (Hq, 1.0))):
        g = torch.Generator(device="cpu")
        g.manual_seed(seed * 10 + i + 1)
        out.append((torch.randn(T, H, D, generator=g, dtype=torch.float32) * s).to(torch.bfloat16))
    return tuple(out)  # Q, K, V, dO


def make_fused_rows(T: int, Hq: int, Hkv: int, D: int, seed: int):
    """bf16 fused projection rows [T, (Hq + 2 Hkv) * D] ~ N(0,1) (the rotary prologue's input) and
    bf16 upstream gradients dQ [T, Hq, D], dK, dV [T, Hkv, D] ~ N(0,1) for its backward."""
    out = []
    for i, shape in enumerate(((T, (Hq + 2 * Hkv) * D), (T, Hq, D), (T, Hkv, D), (T, Hkv, D))):
        g = torch.Generator(device="cpu")
        g.manual_seed(seed * 10 + 5 + i)
        out.append(torch.randn(*shape, generator=g, dtype=torch.float32).to(torch.bfloat16))
    return tuple(out)  # qkv, dQ, dK, dV


def make_layer_tensors(T: int, d_model: int, Hq: int, Hkv: int, D: int, seed: int):
    """bf16 inputs of the segmented layer slice: hidden rows X [T, d_model] ~ N(0,1), the fused
    projection weight W [(Hq + 2 Hkv) D, d_model] ~ N(0,1) / sqrt(d_model) (so that projected
    heads have unit-variance elements), and dO [T, Hq, D] ~ N(0,1)."""
    out = []
    for i, (shape, std) in enumerate((((T, d_model), 1.0),
                                      (((Hq + 2 * Hkv) * D, d_model), 1.0 / math.sqrt(d_model)),
                                      ((T, Hq, D), 1.0))):
        g = torch.Generator(device="cpu")
        g.manual_seed(seed * 10 + 9 + i)
        out.append((torch.randn(*shape, generator=g, dtype=torch.float32) * std).to(torch.bfloat16))
    return tuple(out)  # X, W, dO


def build_case(w: Workload, assign_fn):
    """Lays out a workload: per sequence the full grid of anchors x depths, segments from
    ``assign_fn(anchor, depth, K, boundaries) -> segment per token`` (Algorithm 1, supplied by the
    caller: the library's or the oracle's), tokens ordered by (segment, depth, anchor).
    Returns cu_seqlens, anchor, depth (int32 arrays in memory order) and the partitions as
    dicts {seq, q: (b, e), k: [(b, e), ...]} in execution order."""
    cu = [0]
    anchors, depths, parts = [], [], []
    for i, n in enumerate(w.seq_lens):
        a, d = full_grid(n, w.K) if w.cod_r is None else cod_grid(n, w.K, w.cod_r, w.seed + i)
        bounds = segment_boundaries(n, w.n_segments, w.seg_len)
        if len(bounds) > 2:
            seg = np.asarray(assign_fn(a, d, w.K, bounds), dtype=np.int32)
        else:
            seg = np.zeros(a.shape[0], np.int32)
        perm = arrange_by_segment(a, d, seg, w.order)
        a, d, seg = a[perm], d[perm], seg[perm]
        for p in partitions_from_layout(seg, d, offset=cu[-1]):
            p["seq"] = i
            parts.append(p)
        anchors.append(a)
        depths.append(d)
        cu.append(cu[-1] + a.shape[0])
    return (np.asarray(cu, np.int32), np.concatenate(anchors).astype(np.int32),
            np.concatenate(depths).astype(np.int32), parts)

