"""bnn_mlp_forward_noalloc -- the MLP forward for callers that are not allowed to allocate device memory
(its scratch is an array built into the library).  Checked through the C ABI against the ordinary entry
point, which takes its scratch from a caller-provided workspace, and against the CPU oracle: same scores, on
two calls in a row that share the built-in array.  A workspace that the caller lent to the context for other
calls must come back untouched ("no workspace needed and none used").  This file is collected last on purpose,
so a run that stops at the first failure has already been through every other test; it must also pass when run
on its own in a fresh process."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, nets, workloads as wl

pytestmark = pytest.mark.gpu


def scores_close(got, want):
    # the tolerance of the other MLP tests: 1e-5 relative with an absolute floor for near-zero scores
    got, want = got.astype(np.float64), want.astype(np.float64)
    return bool((np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-6 * np.abs(want).max()).all())


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    build.build()
    ctx = binding.Context(0)
    L = binding.lib()
    limit = int(L.bnn_mlp_noalloc_max_bytes())
    assert limit == 512 * 1024

    # two different problems back to back: the second one is smaller, so stale words of the first remain
    # in the shared array beside it
    runs = [(1024, (784, 4096, 2048, 10), 11), (200, (300, 512, 512, 512, 10), 12)]
    for batch, sizes, seed in runs:
        case = wl.mlp_case(batch=batch, sizes=sizes, seed=seed)
        net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
        X = torch.from_numpy(case["X"]).cuda()

        ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], batch, False), dtype=torch.uint8, device="cuda")
        ctx.set_workspace(ws)
        want = ctx.mlp_forward(net["desc"], X, batch)
        torch.cuda.synchronize()
        ctx.set_workspace(None)                      # from here on the context has no workspace at all
        want_oracle, _ = oracle.mlp_forward(case["X"], case["weights"], case["bns"])

        got = torch.full((batch, sizes[-1]), float("nan"), dtype=torch.float32, device="cuda")
        ctx.mlp_forward_noalloc(net["desc"], X, batch, got)
        torch.cuda.synchronize()
        assert scores_close(got.cpu().numpy(), want.cpu().numpy())
        assert np.array_equal(got.cpu().numpy().argmax(1), want.cpu().numpy().argmax(1))
        assert scores_close(got.cpu().numpy(), want_oracle)
        assert np.array_equal(got.cpu().numpy().argmax(1), want_oracle.argmax(1))

        # the same call while the context holds a workspace lent for other calls: it must not be written
        lent = torch.full((ws.numel(),), 0xA5, dtype=torch.uint8, device="cuda")
        ctx.set_workspace(lent)
        got2 = torch.full((batch, sizes[-1]), float("nan"), dtype=torch.float32, device="cuda")
        ctx.mlp_forward_noalloc(net["desc"], X, batch, got2)
        torch.cuda.synchronize()
        assert bool((lent == 0xA5).all()), "the no-allocation entry point wrote into the caller's workspace"
        assert torch.equal(got2, got)
        ctx.set_workspace(None)

    # a problem beyond the built-in array is refused with its own status and leaves the output alone
    batch, sizes = 1025, (784, 4096, 10)
    case = wl.mlp_case(batch=batch, sizes=sizes, seed=13)
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    out = torch.full((batch, 10), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.BnnError) as e:
        ctx.mlp_forward_noalloc(net["desc"], torch.from_numpy(case["X"]).cuda(), batch, out)
    assert e.value.status == -6
    assert b"built-in scratch" in L.bnn_status_string(-6)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    ctx.close()
