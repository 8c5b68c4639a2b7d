"""GPU: the allocation-free forward entry point against the ordinary one, through the C ABI.

``peagle_attn_fwd_static`` is for callers that cannot call cudaMalloc (a step running inside a
framework whose allocator owns the GPU's memory, a loop that cannot take an allocation's
device-wide synchronisation).  Its tile plan lives in one fixed array inside the library that
every call reuses, so the thing to check is that a call is not disturbed by what the previous
call left there: two calls in a row on different partitions, then the first one again.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import TOL_MAXABS_O, TOL_RELL2_O, DeviceCase, rel_l2

pytestmark = pytest.mark.gpu


def fresh_outputs(case):
    nan = float("nan")
    return torch.full_like(case.O, nan), torch.full_like(case.LSE, nan)


def rows_of(part, O, LSE):
    b, e = part["q"]
    return O[b:e].float().cpu().numpy(), LSE[:, b:e].cpu().numpy()


def assert_matches(got, want):
    (gO, gL), (wO, wL) = got, want
    assert np.isfinite(gO).all()
    finite = np.isfinite(wL)
    assert np.array_equal(np.isneginf(gL), np.isneginf(wL))
    assert np.abs(gO - wO).max() <= TOL_MAXABS_O
    assert np.abs(gL[finite] - wL[finite]).max() <= TOL_MAXABS_O
    assert rel_l2(gO, wO) <= TOL_RELL2_O
    assert rel_l2(gL[finite], wL[finite]) <= TOL_RELL2_O


def test_static_forward_matches_context_forward_on_consecutive_calls():
    # three segments: partitions with one, two and three visible key ranges, ragged tiles
    w = inputs.Workload("no_alloc", (333,), 4, 4, 2, 64, n_segments=3, seed=12)
    case = DeviceCase(w)
    ctx = binding.Context(0)
    try:
        for bp in case.bparts:
            binding.peagle_attn_fwd(ctx, case.prob, bp, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
        assert binding.peagle_poll_status(ctx) == 0
    finally:
        ctx.close()
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda:0")
    # largest partition first, then a smaller one over the leftovers, then the first again
    order = [len(case.parts) - 1, 0, len(case.parts) - 1]
    for i in order:
        O, LSE = fresh_outputs(case)
        binding.peagle_attn_fwd_static(0, case.prob, case.bparts[i], case.dQ_, case.dK_, case.dV_,
                                       O, LSE, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        part = case.parts[i]
        assert_matches(rows_of(part, O, LSE), rows_of(part, case.O, case.LSE))
        b, e = part["q"]                      # rows outside the partition stay untouched
        assert torch.isnan(O[:b].float()).all() and torch.isnan(O[e:].float()).all()


def test_static_forward_rejects_sizes_beyond_its_limit():
    w = inputs.Workload("no_alloc_big", (40,), 2, 2, 1, 64, seed=13)
    case = DeviceCase(w)
    big = binding.Problem(np.array([0, 40000], np.int32), case.d_anchor, case.d_depth, 2, 2, 1, 64,
                          w.scale)
    part = binding.Partition(0, (0, 80))
    with pytest.raises(binding.PeagleError) as err:
        binding.peagle_attn_fwd_static(0, big, part, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
    assert err.value.status == binding.STATUS["TOO_LARGE"]
