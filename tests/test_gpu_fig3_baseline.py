"""The comparison kernel of Fig. 3 (Section 4): a deliberately unoptimized float32 matrix product, fed with +-1 values.
Section 4 says it and the binary kernel return identical outputs on such inputs; here its output is held against the
oracle's integer product (exact in float32: every partial sum is an integer below 2^24)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(300, 200, 1000), (64, 256, 512), (1, 1, 1), (33, 7, 65)])
def test_baseline_kernel_equals_oracle_gemm(M, N, K):
    build.build()
    ctx = binding.Context(0)
    A, B = wl.gemm_case(M, N, K, seed=31)
    C = ctx.baseline_gemm_f32(torch.from_numpy(A).cuda().float(), torch.from_numpy(B).cuda().float())
    torch.cuda.synchronize()
    got = C.cpu().numpy()
    want = oracle.gemm(A, B)
    assert got.dtype == np.float32 and np.array_equal(got, want.astype(np.float32))
    # and the binary kernel on the same inputs returns the same numbers (the statement of Section 4)
    Ap = ctx.pack_signs(torch.from_numpy(A).cuda())
    Bp = ctx.pack_signs(torch.from_numpy(B).cuda(), pack_along=1)
    Cx = ctx.xnor_gemm(Ap, Bp, M, N, K)
    torch.cuda.synchronize()
    assert np.array_equal(Cx.cpu().numpy(), want)
    ctx.close()
