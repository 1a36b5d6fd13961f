"""Exploiting filter repetitions (Section 3.3): with the switch on, bnn_binary_conv2d applies per input channel only the
distinct 2-D 3x3 filters (a filter and its negation count as one) and sums the responses per 3-D filter.  The results
must be the oracle's direct convolution, bit for bit -- on iid weights (nearly all classes occur) and on weights drawn
from a small per-channel dictionary so that about 42 % of a channel's filters are distinct, the share the paper reports
for its trained CIFAR-10 network.  The count of distinct filters is checked against a direct enumeration."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, workloads as wl
from util import np_pack_pm1, np_unpack_pm1, padding_is_zero

pytestmark = pytest.mark.gpu


def count_distinct(wgt):
    Cout, _, _, Cin = wgt.shape
    total = 0
    for c in range(Cin):
        f = wgt[:, :, :, c].reshape(Cout, 9).astype(np.int32)
        f = f * f[:, :1]                                    # a filter and its negation are one class
        total += len({tuple(r) for r in f})
    return total


@pytest.mark.parametrize("B,H,W,Cin,Cout,pool,kind", [(2, 8, 8, 32, 40, False, "iid"), (3, 6, 10, 64, 130, True, "iid"),
                                                      (2, 16, 16, 128, 128, True, "dict"), (1, 5, 7, 32, 128, False, "dict"),
                                                      (1, 1, 1, 32, 33, False, "iid")])
def test_filter_repetition_conv_matches_oracle(B, H, W, Cin, Cout, pool, kind):
    build.build()
    ctx = binding.Context(0)
    rng = np.random.default_rng(B * 1000 + Cin + Cout)
    act = wl.pm1(rng, (B, H, W, Cin))
    distinct = max(1, int(round(0.42 * Cout)))
    wgt = wl.pm1(rng, (Cout, 3, 3, Cin)) if kind == "iid" else wl.dictionary_conv_weights(rng, Cout, Cin, min(distinct, 256))
    S = oracle.conv3x3(act, wgt)
    thr = rng.integers(-20, 21, Cout).astype(np.int32)
    thr[0] = S[0, 0, 0, 0]                       # a tie on a corner pixel
    flip = rng.integers(0, 2, Cout).astype(np.uint8)
    P = oracle.maxpool2x2(S) if pool else S
    want = oracle.threshold(P, thr, flip)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    actp = dev(np_pack_pm1(act).view(np.int32))
    Wp = dev(np_pack_pm1(wgt.reshape(Cout, 9, Cin)).reshape(Cout, -1).view(np.int32))
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    ws = torch.empty(ctx.filter_repetition_workspace_bytes(Cin, Cout), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    assert ctx.filter_repetition_count(Wp, Cin, Cout) == count_distinct(wgt)
    if kind == "dict":
        assert ctx.filter_repetition_count(Wp, Cin, Cout) == min(distinct, 256) * Cin
    ctx.set_conv_filter_repetition(True)
    bits, sums = ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p, want_sums=True)
    torch.cuda.synchronize()
    assert np.array_equal(sums.cpu().numpy(), P)
    got = bits.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, Cout), want)
    assert padding_is_zero(got, Cout)
    # and without the switch the same call gives the same words
    ctx.set_conv_filter_repetition(False)
    bits2, _ = ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p)
    torch.cuda.synchronize()
    assert torch.equal(bits2, bits)
    ctx.set_workspace(None)
    ctx.set_conv_filter_repetition(True)
    with pytest.raises(binding.BnnError) as e:
        ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p)
    assert e.value.status == -3
    ctx.close()
