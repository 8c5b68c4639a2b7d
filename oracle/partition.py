"""TEST INFRASTRUCTURE: the paper's Algorithm 1 (sequence partitioning) and the COD position
count, written out plainly in Python.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA library has its own host code.

Notation follows Algorithm 1: P[g] is the set of sequence positions p kept at depth g (a token
(anchor a, depth g) sits at position p = a + g), S the number of segments, L the sequence
length, B the boundaries, A[g][p] the segment of position p at depth g, N[s] the depth-0
positions segment s may see.
"""
from __future__ import annotations


def boundaries(L: int, S: int) -> list[int]:
    """Algorithm 1, initialisation: B = {0, L/S, 2L/S, ..., L} (floor where S does not divide L)."""
    return [(k * L) // S for k in range(S + 1)]


def assign_segments(P: list[list[int]], S: int, L: int, B: list[int] | None = None):
    """Algorithm 1.  Returns (A, N, B).  ``B`` overrides the even boundaries (used where a
    workload fixes the segment length instead of the segment count)."""
    B = boundaries(L, S) if B is None else list(B)
    assert len(B) == S + 1 and B[0] == 0 and B[-1] == L
    A: list[dict[int, int]] = [dict() for _ in P]
    # Phase 1: depths 0 and 1 by position index.  A position at or past L (the last anchors'
    # chains reach there) would get segment S; it is kept in the last segment.
    for g in range(min(2, len(P))):
        for p in P[g]:
            s = max(s for s in range(S + 1) if B[s] <= p)
            A[g][p] = min(s, S - 1)
    # Phase 2: deeper positions inherit the segment of their dependency (p-1 at depth g-1).
    for g in range(2, len(P)):
        for p in P[g]:
            A[g][p] = A[g - 1][p - 1]
    # Phase 3: depth-0 positions visible to segment s, cumulative up to its boundary.
    N = [[p for p in P[0] if p < B[s + 1]] for s in range(S)]
    return A, N, B


def cod_total_positions(n: int, K: int, r: float) -> float:
    """Section 3.2: total positions with retention rate r, n (1 - r^K) / (1 - r)."""
    return n * (1.0 - r ** K) / (1.0 - r)
