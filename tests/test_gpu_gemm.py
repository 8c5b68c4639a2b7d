"""GPU: the projection products (peagle_gemm_bf16) against fp64 matrix products of the same
bf16-rounded operands, through the C ABI: the four operand layouts, ragged sizes in every
dimension, sub-matrices with a leading dimension, and the fp32 accumulate mode."""
import numpy as np
import pytest
import torch

from paper_2602_01469_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g).to(torch.bfloat16)


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (200, 264, 200), (1, 8, 8), (513, 1024, 2880), (300, 72, 1000),
                                   (300, 1160, 520),   # wide tiles with a ragged last column of tiles
                                   (200, 1024, 136)])  # one pair of CTAs whose second CTA holds 72 rows
@pytest.mark.parametrize("a_t,b_t", [(0, 0), (0, 1), (1, 1), (1, 0)])
def test_products_match_fp64(ctx, M, N, K, a_t, b_t):
    def pad8(x):
        return (x + 7) // 8 * 8
    # operands live inside larger buffers: leading dimensions differ from the extents
    A = rand_bf16((K, pad8(M) + 8) if a_t else (M, pad8(K) + 16), 1)
    B = rand_bf16((K, pad8(N) + 8) if b_t else (N, pad8(K) + 8), 2)
    Av = (A[:, :M].t() if a_t else A[:, :K]).double()
    Bv = (B[:, :N].t() if b_t else B[:, :K]).double()
    want = (Av @ Bv.t()).numpy()
    dA, dB = A.cuda(), B.cuda()
    ldc = pad8(N) + 8
    C = torch.full((M, ldc), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.peagle_gemm_bf16(ctx, dA, A.shape[1], a_t, dB, B.shape[1], b_t, C, ldc, 0, M, N, K)
    assert binding.peagle_poll_status(ctx) == 0
    got = C[:, :N].float().cpu().numpy()
    assert torch.isnan(C[:, N:].float()).all()                 # nothing outside M x N is written
    scale = np.abs(want).max()
    assert np.abs(got - want).max() <= 2.0 ** -8 * scale + 1e-6      # one bf16 rounding of the result
    # fp32 accumulate: two calls add twice, on top of what was there
    Cf = torch.ones((M, ldc), dtype=torch.float32, device="cuda")
    for _ in range(2):
        binding.peagle_gemm_bf16(ctx, dA, A.shape[1], a_t, dB, B.shape[1], b_t, Cf, ldc, 1, M, N, K)
    assert binding.peagle_poll_status(ctx) == 0
    gotf = Cf[:, :N].cpu().numpy()
    assert np.abs(gotf - (1.0 + 2.0 * want)).max() <= 1e-4 * max(scale, 1.0) * max(1.0, K / 256)
    assert torch.all(Cf[:, N:] == 1.0)
