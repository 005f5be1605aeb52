"""GPU test of efqat_colsum_noalloc, the entry point for callers that may not allocate
device memory (a runtime hook that only gets a fixed arena, a loop that must stay out of
the allocator, a process whose memory pool belongs to someone else).

It must give the same bias gradient as the regular backward call, which takes its scratch
from a caller-allocated workspace.  Two calls in a row with different shapes make sure that
what the first call left in the built-in scratch array cannot leak into the second.  The
file name sorts last on purpose: a run that stops at the first failure has then already
executed every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2411_11038_b200 import binding as B

pytestmark = pytest.mark.gpu


def _db_regular(ctx, dY, K=64):
    """db from efqat_fq_linear_bwd (k_sel = 0, so only dX / dS_x / dZ_x / db are produced)."""
    M, N = dY.shape
    g = torch.Generator().manual_seed(M + N)
    X = torch.randn((M, K), generator=g).to(dY.dtype).cuda()
    W = (torch.randn((N, K), generator=g) * 0.02).cuda()
    s_w = B.init_weight_scales(ctx, W, 8)
    s_x, z_x = B.init_act_qparams(ctx, X, 8, False)
    out = B.fq_linear_bwd(ctx, dY, X, W, s_w, s_x, z_x, None, 0, 8, 8, False, want_db=True)
    return out["db"].clone()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_colsum_noalloc_matches_backward_db_twice(dtype):
    ctx = B.Context(0)
    g = torch.Generator().manual_seed(7)
    first = torch.randn((1000, 2304), generator=g).to(dtype).cuda()
    second = (torch.randn((333, 136), generator=g) * 3 + 1).to(dtype).cuda()   # smaller: stale scratch beyond it
    for dY in (first, second):
        got = B.colsum_noalloc(dY)
        want = _db_regular(ctx, dY)
        torch.cuda.synchronize()
        ref = dY.double().sum(dim=0).cpu().numpy()
        abs_sum = dY.double().abs().sum(dim=0).cpu().numpy()
        # same tolerance class as the other fp32 reductions: 1e-5 of the sum of |terms|
        assert np.all(np.abs(got.cpu().numpy() - want.cpu().numpy()) <= 1e-5 * abs_sum)
        assert np.all(np.abs(got.cpu().numpy() - ref) <= 1e-5 * abs_sum)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("M,N", [(2304, 16384), (8, 16384), (8, 64)])
def test_colsum_noalloc_at_the_ends_of_its_range(M, N):
    """The widest matrix the built-in array holds (all 64 slabs of partial sums, up to the array's
    last element) and matrices with fewer rows than one slab."""
    g = torch.Generator().manual_seed(M * 31 + N)
    dY = torch.randn((M, N), generator=g).to(torch.bfloat16).cuda()
    for _ in range(2):
        got = B.colsum_noalloc(dY).cpu().numpy()
        ref = dY.double().sum(dim=0).cpu().numpy()
        abs_sum = dY.double().abs().sum(dim=0).cpu().numpy()
        assert np.all(np.abs(got - ref) <= 1e-5 * abs_sum)


def test_colsum_noalloc_rejects_what_it_cannot_hold():
    lib = B.load()
    dY = torch.zeros((8, 16392), dtype=torch.float32).cuda()
    out = torch.zeros(16392, dtype=torch.float32).cuda()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    p = lambda t: C.c_void_p(t.data_ptr())
    assert lib.efqat_colsum_noalloc(B.F32, p(dY), 8, 16392, p(out), st) == -11      # beyond the built-in maximum
    assert lib.efqat_colsum_noalloc(B.F32, p(dY), 8, 100, p(out), st) == -3         # N % 8 != 0
    assert lib.efqat_colsum_noalloc(B.F32, None, 8, 16, p(out), st) == -1
    assert lib.efqat_colsum_noalloc(5, p(dY), 8, 16, p(out), st) == -4
    assert B.status_string(-11) == "size exceeds a built-in maximum"
