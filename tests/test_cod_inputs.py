"""CPU: the COD-subsampled metadata generator (Section 3's geometric decay, Section 3.2's nesting)
and what the oracle's Algorithm 1 and mask make of its output."""
import numpy as np
import pytest

from oracle import partition as opart
from oracle import peagle_oracle as orc
from paper_2602_01469_b200 import inputs


@pytest.mark.parametrize("n,K,r", [(8192, 8, 0.8), (1000, 5, 0.7), (16, 4, 0.7)])
def test_cod_counts_follow_the_geometric_decay(n, K, r):
    a, d = inputs.cod_grid(n, K, r, seed=3)
    counts = [int((d == g).sum()) for g in range(K)]
    assert counts[0] == n
    for g in range(1, K):
        assert abs(counts[g] - n * r ** g) <= g + 1 + (g if n < 100 else 0)  # rounding, end clipping
    if n >= 1000:                                        # Section 3.2: n (1 - r^K) / (1 - r)
        assert abs(sum(counts) - opart.cod_total_positions(n, K, r)) <= K


def test_cod_sets_are_nested_along_chains_and_stay_inside_the_sequence():
    n, K = 500, 6
    a, d = inputs.cod_grid(n, K, 0.75, seed=9)
    have = set(zip(a.tolist(), d.tolist()))
    assert len(have) == a.shape[0]                       # no duplicates
    for (x, g) in have:
        assert x + g < n                                 # position p = anchor + depth exists
        if g > 0:
            assert (x, g - 1) in have                    # p-1 at depth g-1 was kept
    other = inputs.cod_grid(n, K, 0.75, seed=10)[0]      # another example draws other positions
    assert other.shape != a.shape or not np.array_equal(other, a)


def test_algorithm_1_and_the_mask_on_cod_metadata():
    n, K, S = 300, 5, 3
    a, d = inputs.cod_grid(n, K, 0.7, seed=4)
    P = inputs.position_sets(a, d, K)
    A, N, B = opart.assign_segments(P, S, n)
    for g in range(2, K):                                # a position and its dependency share a segment
        for p in P[g]:
            assert A[g][p] == A[g - 1][p - 1]
    m = orc.mask_dense(a, d)
    # every token sees the real context up to its anchor and its own chain, nothing else
    assert int(m.sum()) == int(a.astype(np.int64).sum() + d.astype(np.int64).sum() + a.shape[0])
