"""GPU: the rotary prologue and its backward, through the C ABI, against the fp64 oracle.

bf16 inputs, cos / sin from an fp64 angle, fp32 arithmetic, bf16 outputs: an output is the exact
value rounded once to bf16, give or take the rare value that sits on a rounding boundary, plus the
fp32 rounding of x cos - y sin, which is relative to |x| + |y| and so shows where the two products
cancel.  The bar per element is therefore one bf16 unit in the last place (2^-8 relative) plus
1e-5 absolute (inputs are N(0, 1): |x| + |y| < 12, times a few fp32 roundings of 2^-24), with
nearly all elements equal to the rounded oracle value bit for bit; copied value heads are
bit-exact.
"""
import numpy as np
import pytest
import torch

from oracle import rope_oracle as ro
from paper_2602_01469_b200 import binding, inputs

pytestmark = pytest.mark.gpu

BASE = 500000.0
DEV = "cuda:0"


def positions(T, K, n, seed):
    """anchor, depth of a depth-major grid cut to T tokens, shuffled so that neighbours differ."""
    a, d = inputs.full_grid(n, K)
    idx = np.random.default_rng(seed).permutation(a.shape[0])[:T]
    return a[idx].astype(np.int32), d[idx].astype(np.int32)


def check(got_bf16, want64):
    got = got_bf16.float().cpu().numpy().astype(np.float64)
    ulp = np.abs(want64) * 2.0 ** -8 + 1e-5
    assert np.all(np.abs(got - want64) <= ulp), float(np.max(np.abs(got - want64) / ulp))
    rounded = torch.from_numpy(want64).to(torch.bfloat16).float().numpy()
    assert np.mean(rounded == got) > 0.999


@pytest.mark.parametrize("T,Hq,Hkv,D,n,K", [
    (301, 4, 2, 64, 20000, 8),     # ragged token count, positions up to 2e4
    (130, 6, 2, 128, 4096, 4),
    (1, 1, 1, 64, 10, 2),
    (2051, 64, 8, 64, 4096, 8),    # the headline head counts, several blocks
])
def test_forward_and_backward_match_the_oracle(T, Hq, Hkv, D, n, K):
    ctx = binding.Context(0)
    anchor, depth = positions(T, K, n, seed=T)
    qkv, gQ, gK, gV = inputs.make_fused_rows(T, Hq, Hkv, D, seed=T)
    d_anchor, d_depth = torch.from_numpy(anchor).to(DEV), torch.from_numpy(depth).to(DEV)
    nan = float("nan")
    Q = torch.full((T, Hq, D), nan, dtype=torch.bfloat16, device=DEV)
    K_ = torch.full((T, Hkv, D), nan, dtype=torch.bfloat16, device=DEV)
    V = torch.full((T, Hkv, D), nan, dtype=torch.bfloat16, device=DEV)
    binding.peagle_rope_qkv_fwd(ctx, qkv.to(DEV), d_anchor, d_depth, Hq, Hkv, D, BASE, Q, K_, V)
    torch.cuda.synchronize()
    wQ, wK, wV = ro.rope_qkv_fwd(qkv.float().numpy(), anchor, depth, Hq, Hkv, D, BASE)
    check(Q, wQ)
    check(K_, wK)
    assert torch.equal(V.cpu(), qkv[:, (Hq + Hkv) * D:].reshape(T, Hkv, D))

    gx = torch.full((T, (Hq + 2 * Hkv) * D), nan, dtype=torch.bfloat16, device=DEV)
    binding.peagle_rope_qkv_bwd(ctx, gQ.to(DEV), gK.to(DEV), gV.to(DEV), d_anchor, d_depth, Hq, Hkv,
                                D, BASE, gx)
    torch.cuda.synchronize()
    want = ro.rope_qkv_bwd(gQ.float().numpy(), gK.float().numpy(), gV.float().numpy(), anchor, depth,
                           Hq, Hkv, D, BASE)
    check(gx, want)
    assert torch.equal(gx[:, (Hq + Hkv) * D:].cpu(), gV.reshape(T, Hkv * D))
    assert binding.peagle_poll_status(ctx) == 0


def test_headline_shape_sampled_rows():
    """n = 4096, K = 8, 64 / 8 heads of 64: every token on the device, 256 sampled rows checked."""
    w = inputs.WORKLOADS[inputs.HEADLINE]
    ctx = binding.Context(0)
    anchor, depth = inputs.full_grid(w.seq_lens[0], w.K)
    T, Hq, Hkv, D = anchor.shape[0], w.n_q_heads, w.n_kv_heads, w.head_dim
    qkv = inputs.make_fused_rows(T, Hq, Hkv, D, seed=w.seed)[0]
    Q = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=DEV)
    K_ = torch.empty((T, Hkv, D), dtype=torch.bfloat16, device=DEV)
    V = torch.empty((T, Hkv, D), dtype=torch.bfloat16, device=DEV)
    binding.peagle_rope_qkv_fwd(ctx, qkv.to(DEV), torch.from_numpy(anchor).to(DEV),
                                torch.from_numpy(depth).to(DEV), Hq, Hkv, D, BASE, Q, K_, V)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(0).choice(T, 256, replace=False))
    wQ, wK, _ = ro.rope_qkv_fwd(qkv[rows].float().numpy(), anchor[rows], depth[rows], Hq, Hkv, D, BASE)
    check(Q[rows], wQ)
    check(K_[rows], wK)
    assert torch.equal(V.cpu().reshape(T, -1), qkv[:, (Hq + Hkv) * D:])


def test_empty_and_rejected_arguments():
    ctx = binding.Context(0)
    z = torch.zeros((0, 6 * 64), dtype=torch.bfloat16, device=DEV)
    zi = torch.zeros(0, dtype=torch.int32, device=DEV)
    out = torch.zeros((1, 64), dtype=torch.bfloat16, device=DEV)
    binding.peagle_rope_qkv_fwd(ctx, z, zi, zi, 4, 1, 64, BASE, out, out, out)  # no tokens: nothing runs
    torch.cuda.synchronize()
    assert float(out.abs().sum()) == 0.0
    with pytest.raises(binding.PeagleError):
        binding.peagle_rope_qkv_fwd(ctx, out, zi, zi, 4, 1, 96, BASE, out, out, out)
    with pytest.raises(binding.PeagleError):
        binding.peagle_rope_qkv_fwd(ctx, out, zi, zi, 4, 1, 64, 1.0, out, out, out)
