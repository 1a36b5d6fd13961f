"""A reduction longer than 2^24: sums of +-1 are then no longer exact in the float32 accumulators of the 4-bit tensor
path, so the library must take byte operands with int32 accumulators instead.  256 x 128 outputs over K = 2^24 + 32:
sampled rows against the oracle, every output against the library product, plus the invariants that hold for
any +-1 product (same parity as K, magnitude at most K)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build

pytestmark = pytest.mark.gpu


def test_reduction_longer_than_2_to_24_uses_exact_accumulators():
    psutil = pytest.importorskip("psutil")
    if psutil.virtual_memory().available < 24 << 30 or torch.cuda.mem_get_info()[0] < 32 << 30:
        pytest.skip("needs about 8 GB of host and 16 GB of device memory")
    build.build()
    ctx = binding.Context(0)
    M, N, K = 256, 128, (1 << 24) + 32
    g = torch.Generator(device="cuda").manual_seed(51)
    A = torch.randint(0, 2, (M, K), device="cuda", generator=g, dtype=torch.int8) * 2 - 1
    Bt = torch.randint(0, 2, (N, K), device="cuda", generator=g, dtype=torch.int8) * 2 - 1      # B transposed: N x K
    # make two rows extreme, so that sums far beyond 2^24 occur as well: row 0 = column 0 of B, row 1 = its negation
    A[0] = Bt[0]
    A[1] = -Bt[0]
    Ap = ctx.pack_signs(A)
    Bp = ctx.pack_signs(Bt)                                      # already K-major: packed like A
    ws = torch.empty(ctx.gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    assert ws.numel() > 0
    ctx.set_workspace(ws)
    ctx.set_engine(binding.ENGINE_TENSOR)
    C = ctx.xnor_gemm(Ap, Bp, M, N, K)
    ctx.device_status()
    assert int(C[0, 0]) == K and int(C[1, 0]) == -K
    assert bool(((C - K) % 2 == 0).all()) and int(C.abs().max()) <= K
    # every output against the library product, in slices of 2^20 along K (each slice is exact in float32)
    torch.backends.cuda.matmul.allow_tf32 = False
    ref = torch.zeros(M, N, dtype=torch.int64, device="cuda")
    for k0 in range(0, K, 1 << 20):
        ref += torch.matmul(A[:, k0:k0 + (1 << 20)].float(), Bt[:, k0:k0 + (1 << 20)].float().t()).to(torch.int64)
    assert torch.equal(C.to(torch.int64), ref)
    rows = np.array([0, 1, 2, 127, 128, 255])
    want = oracle.gemm(A[torch.from_numpy(rows).cuda()].cpu().numpy(), np.ascontiguousarray(Bt.cpu().numpy().T))
    assert np.array_equal(C[torch.from_numpy(rows).cuda()].cpu().numpy(), want)
    # the CUDA-core kernel on the same operands
    ctx.set_engine(binding.ENGINE_POPC)
    C1 = ctx.xnor_gemm(Ap, Bp, M, N, K)
    torch.cuda.synchronize()
    assert torch.equal(C1, C)
    ctx.set_workspace(None)
    ctx.close()
