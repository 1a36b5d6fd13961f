"""The tensor-core kernels wait on barriers with a bound.  Here one such wait is made to run out, with nothing on the GPU
faulting, trapping or hanging: a host-side switch makes the producer of the single-SM kernel request no operands, so the
warps that would consume them give up after the (shortened) limit, the kernel frees its tensor memory and ends, the
context reports BNN_ERR_DEVICE_STATUS once, and the next ordinary call on the same context is exact again.
The CTA-pair form of the kernel shares the waiting code but is not driven into its failure path on the GPU."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [8, 4])
def test_bounded_wait_runs_out_and_context_stays_usable(bits):
    build.build()
    ctx = binding.Context(0)
    ctx.set_engine(binding.ENGINE_TENSOR)
    ctx.set_operand_bits(bits)
    M, N, K = 256, 128, 256
    A, B = wl.gemm_case(M, N, K, seed=41)
    Ap = ctx.pack_signs(torch.from_numpy(A).cuda())
    Bp = ctx.pack_signs(torch.from_numpy(B).cuda(), pack_along=1)
    A_exp = (ctx.expand_signs_f4 if bits == 4 else ctx.expand_signs)(Ap, M, K)
    B_exp = (ctx.expand_signs_f4 if bits == 4 else ctx.expand_signs)(Bp, N, K)
    thr = torch.zeros(N, dtype=torch.int32, device="cuda")
    want = oracle.threshold(oracle.gemm(A, B), np.zeros(N, np.int32))

    def run():
        out, _ = ctx.binary_dense_expanded(A_exp, B_exp, bits, thr, None, M, N, K)
        return out

    from util import np_unpack_pm1
    good = run()
    ctx.device_status()
    assert np.array_equal(np_unpack_pm1(good.cpu().numpy(), N), want)

    ctx.set_wait_limit_ns(5_000_000)          # 5 ms
    ctx.debug_drop_loads(True)
    t0 = time.perf_counter()
    run()                                      # returns: the kernel gives up and runs to its normal end
    with pytest.raises(binding.BnnError) as e:
        ctx.device_status()
    elapsed = time.perf_counter() - t0
    assert e.value.status == -5
    assert elapsed < 1.0, "one failure should cost about one limit, not one per waiter"
    ctx.device_status()                        # reported once, then clear

    ctx.debug_drop_loads(False)
    ctx.set_wait_limit_ns(2_000_000_000)
    again = run()
    ctx.device_status()
    assert torch.equal(again, good)
    ctx.close()
