"""CPU-only checks of the library's host side: the shared object loads and exports every symbol
the header declares, and its Algorithm 1 agrees with the oracle's."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import partition as opart
from paper_2602_01469_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "peagle.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(peagle_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for name, code in binding.STATUS.items():
        assert lib.peagle_status_string(code).decode() != "unknown status", name
    assert lib.peagle_status_string(-99).decode() == "unknown status"


def oracle_segments(anchor, depth, K, bounds):
    P = inputs.position_sets(anchor, depth, K)
    A, N, B = opart.assign_segments(P, len(bounds) - 1, bounds[-1], B=bounds)
    return np.array([A[d][a + d] for a, d in zip(anchor, depth)], np.int32)


@pytest.mark.parametrize("n,K,S", [(16, 4, 2), (37, 5, 4), (11008 // 8, 8, 4), (64, 1, 3), (5, 8, 5)])
def test_assign_segments_matches_oracle_full_grid(lib, n, K, S):
    anchor, depth = inputs.full_grid(n, K)
    rng = np.random.default_rng(0)
    perm = rng.permutation(n * K)
    anchor, depth = anchor[perm], depth[perm]
    bounds = inputs.segment_boundaries(n, S)
    got = binding.peagle_assign_segments(anchor, depth, K, bounds)
    assert np.array_equal(got, oracle_segments(anchor, depth, K, bounds))


def test_assign_segments_fig3_example(lib):
    P = []
    for line in open(os.path.join(ROOT, "tests", "golden", "fig3_cod_example.txt")):
        if line.startswith("depth"):
            P.append([int(x) for x in line.split(":")[1].split()])
    anchor = np.array([p - g for g, ps in enumerate(P) for p in ps], np.int32)
    depth = np.array([g for g, ps in enumerate(P) for _ in ps], np.int32)
    got = binding.peagle_assign_segments(anchor, depth, 4, [0, 8, 16])
    assert np.array_equal(got, oracle_segments(anchor, depth, 4, [0, 8, 16]))
    tok = {(int(a), int(d)): int(s) for a, d, s in zip(anchor, depth, got)}
    assert tok[(6, 2)] == tok[(6, 1)] == 0          # position 8 depth 2 with position 7 depth 1


def test_assign_segments_fixed_length_boundaries(lib):
    n, K = 300, 4
    anchor, depth = inputs.full_grid(n, K)
    bounds = inputs.segment_boundaries(n, seg_len=128)
    assert bounds == [0, 128, 256, 300]
    got = binding.peagle_assign_segments(anchor, depth, K, bounds)
    assert np.array_equal(got, oracle_segments(anchor, depth, K, bounds))


def test_assign_segments_rejects_missing_dependency_and_bad_args(lib):
    with pytest.raises(binding.PeagleError) as e:
        binding.peagle_assign_segments([0, 1, 1], [0, 0, 2], 3, [0, 2])   # (1,2) without (1,1)
    assert e.value.status == binding.STATUS["BAD_META"]
    with pytest.raises(binding.PeagleError) as e:
        binding.peagle_assign_segments([0, 5], [0, 0], 1, [0, 2])         # anchor beyond n
    assert e.value.status == binding.STATUS["BAD_META"]
    with pytest.raises(binding.PeagleError) as e:
        binding.peagle_assign_segments([0], [0], 1, [1, 2])               # boundaries[0] != 0
    assert e.value.status == binding.STATUS["BAD_RANGE"]


def test_build_case_layout_and_partitions(lib):
    w = inputs.Workload("t", (50, 7), 3, 2, 1, 64, n_segments=3)
    cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
    assert cu.tolist() == [0, 150, 171]
    assert sum(p["q"][1] - p["q"][0] for p in parts) == 171
    for p in parts:
        b, e = cu[p["seq"]], cu[p["seq"] + 1]
        assert b <= p["q"][0] < p["q"][1] <= e
        assert all(b <= kb < ke <= e for kb, ke in p["k"])
        assert p["k"][-1][1] == p["q"][1]           # own block is the last visible range


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()
