"""GPU: the allocation-free forward entry point against the fp64 oracle, through the C ABI.

``peagle_attn_fwd_static`` is for callers that cannot call cudaMalloc (a step running inside a
framework whose allocator owns the GPU's memory, a loop that cannot take an allocation's
device-wide synchronisation).  Its tile plan lives in one fixed array inside the library that
every call reuses, so the things to check are: its results are right (against the oracle, and
equal to the ordinary entry point's), a call is not disturbed by what the previous call left in
the array (two calls in a row on different partitions, then the first one again), it really
allocates nothing (free device memory is unchanged across a call), and it works at the largest
shape it accepts.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding, inputs
from tests.gpu_common import DeviceCase, check_forward

pytestmark = pytest.mark.gpu


def fresh_outputs(case):
    nan = float("nan")
    return torch.full_like(case.O, nan), torch.full_like(case.LSE, nan)


def rows_of(part, O, LSE):
    """O [rows][H][D], LSE [rows][H] of a partition's query rows."""
    b, e = part["q"]
    return O[b:e].float().cpu().numpy(), LSE[:, b:e].t().cpu().numpy()


def test_static_forward_matches_oracle_and_context_forward_on_consecutive_calls():
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
    want = [case.oracle_fwd(p) for p in case.parts]
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda:0")
    # largest partition first, then a smaller one over the leftovers, then the first again
    order = [len(case.parts) - 1, 0, len(case.parts) - 1]
    for n_call, i in enumerate(order):
        O, LSE = fresh_outputs(case)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(0)[0]
        binding.peagle_attn_fwd_static(0, case.prob, case.bparts[i], case.dQ_, case.dK_, case.dV_,
                                       O, LSE, status)
        torch.cuda.synchronize()
        if n_call > 0:       # the first call on a device may load the kernels' code
            assert torch.cuda.mem_get_info(0)[0] == free_before, "the call allocated device memory"
        assert int(status.item()) == 0
        part = case.parts[i]
        gO, gL = rows_of(part, O, LSE)
        check_forward(gO, gL, *want[i])                       # against the fp64 oracle
        cO, cL = rows_of(part, case.O, case.LSE)              # and the same bits as the context path
        assert np.array_equal(gO, cO) and np.array_equal(gL, cL)
        b, e = part["q"]                      # rows outside the partition stay untouched
        assert torch.isnan(O[:b].float()).all() and torch.isnan(O[e:].float()).all()
    # without a status word: same result (device-side errors would go unreported)
    O, LSE = fresh_outputs(case)
    binding.peagle_attn_fwd_static(0, case.prob, case.bparts[0], case.dQ_, case.dK_, case.dV_, O, LSE,
                                   None)
    torch.cuda.synchronize()
    check_forward(*rows_of(case.parts[0], O, LSE), *want[0])


def test_static_forward_at_its_limit_shape():
    """The largest call it accepts: 32,768 tokens, 256 x 256 tiles (the headline grid), sampled
    rows against the oracle."""
    w = inputs.WORKLOADS["gptoss_n4096"]
    case = DeviceCase(w)
    assert case.T == 32768
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    O, LSE = fresh_outputs(case)
    binding.peagle_attn_fwd_static(0, case.prob, case.bparts[0], case.dQ_, case.dK_, case.dV_, O, LSE,
                                   status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    rng = np.random.default_rng(2)
    rows = np.unique(np.concatenate([[0, case.T - 1], rng.integers(0, case.T, size=24)]))
    wO, wL = case.oracle_fwd(case.parts[0], rows=rows)
    rt = torch.as_tensor(rows, device="cuda")
    check_forward(O[rt].float().cpu().numpy(), LSE[:, rt].t().cpu().numpy(), wO, wL)


def test_static_forward_rejects_sizes_beyond_its_limit():
    w = inputs.Workload("no_alloc_big", (40,), 2, 2, 1, 64, seed=13)
    case = DeviceCase(w)
    big = binding.Problem(np.array([0, 40000], np.int32), case.d_anchor, case.d_depth, 2, 2, 1, 64,
                          w.scale)
    part = binding.Partition(0, (0, 80))
    with pytest.raises(binding.PeagleError) as err:
        binding.peagle_attn_fwd_static(0, big, part, case.dQ_, case.dK_, case.dV_, case.O, case.LSE)
    assert err.value.status == binding.STATUS["TOO_LARGE"]
