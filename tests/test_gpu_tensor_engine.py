"""GPU parity of the tensor-core engine (int8 tcgen05 path) against the oracle: the same calls as the
CUDA-core path, forced onto the tensor engine through bnn_set_engine, on shapes that span several
128 x 256 tiles with ragged edges in M, N and K."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, nets, workloads as wl
from util import np_pack_pm1, np_unpack_pm1, padding_is_zero

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[(2, 8), (1, 8), (1, 4), (2, 4)],
                ids=["pairs-bytes", "single-bytes", "nibbles", "pairs-nibbles"])
def ctx(request):
    """Tensor engine forced: byte operands with CTA pairs (cta_group::2) wherever the kernel allows, byte operands on
    the single-SM kernel, and 4-bit (e2m1) operands for the +-1 x +-1 products."""
    build.build()
    c = binding.Context(0)
    c.set_engine(binding.ENGINE_TENSOR)
    c.set_pair_mode(request.param[0])
    c.set_operand_bits(request.param[1])
    yield c
    torch.cuda.synchronize()
    c.close()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t if dtype is None else t.to(dtype)).cuda()


def with_ws(ctx, nbytes):
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    return ws


@pytest.mark.parametrize("M,N,K", [(1000, 1100, 1000), (300, 4096, 1024), (512, 640, 4100), (257, 129, 32768),
                                   (2048, 2048, 2048), (1111, 512, 2100), (513, 300, 7000), (3000, 1024, 400)])
def test_xnor_gemm_tensor_engine(ctx, M, N, K):
    A, B = wl.gemm_case(M, N, K, seed=M + N + K)
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Bp = ctx.pack_signs(dev(B, torch.int8), pack_along=1)
    need = ctx.gemm_workspace_bytes(M, N, K)
    assert need > 0
    with pytest.raises(binding.BnnError) as e:          # forced engine without workspace is an error, not a fallback
        ctx.set_workspace(None)
        ctx.xnor_gemm(Ap, Bp, M, N, K)
    assert e.value.status == -3
    ws = with_ws(ctx, need)
    if K % 32:
        Ap[:, K // 32] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")   # garbage in the padding
        Bp[:, K // 32] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")
    ldc = N + 3
    big = torch.full((M + 2, ldc), 12345, dtype=torch.int32, device="cuda")
    ctx.xnor_gemm(Ap, Bp, M, N, K, C=big[1:], ldc=ldc)
    ctx.device_status()
    out = big.cpu().numpy()
    assert np.array_equal(out[1:M + 1, :N], oracle.gemm(A, B))
    assert (out[0] == 12345).all() and (out[M + 1] == 12345).all() and (out[:, N:] == 12345).all()
    ctx.set_workspace(None)
    del ws


@pytest.mark.parametrize("M,N,K", [(700, 1500, 1000), (1000, 4096, 300), (300, 130, 30000)])
def test_binary_dense_tensor_engine(ctx, M, N, K):
    rng = np.random.default_rng(M + N)
    A, W = wl.gemm_case(M, N, K, seed=M * N)
    S = oracle.gemm(A, W)
    thr = rng.integers(-40, 41, N).astype(np.int32)
    d = min(M, N)
    thr[:d] = S[np.arange(d), np.arange(d)]            # exact ties
    thr[-1], thr[-2] = K + 1, -K
    flip = rng.integers(0, 2, N).astype(np.uint8)
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    ws = with_ws(ctx, ctx.gemm_workspace_bytes(M, N, K))
    ld = binding.packed_ld(N) + 4
    out = torch.full((M, ld), -1, dtype=torch.int32, device="cuda")
    ctx.binary_dense(Ap, Wp, dev(thr), flip_p, M, N, K, out=out, ldo_w=ld)
    ctx.device_status()
    got = out.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, N), oracle.threshold(S, thr, flip))
    assert padding_is_zero(got, N)
    ctx.set_workspace(None)
    del ws


@pytest.mark.parametrize("M,N,K", [(700, 2048, 784), (1300, 1000, 784), (600, 2000, 1008)])
def test_first_layer_tensor_engine(ctx, M, N, K):
    rng = np.random.default_rng(M)
    X = wl.u8(rng, (M, K))
    X[0, :] = 255
    X[1, :] = 0
    W = wl.pm1(rng, (K, N))
    S = oracle.first_layer(X, W)
    thr = rng.integers(-3000, 3000, N).astype(np.int32)
    thr[0] = S[0, 0]
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    ws = with_ws(ctx, ctx.gemm_workspace_bytes(M, N, K))
    bits, sums = ctx.first_layer_bitplanes(dev(X), Wp, M, N, K, thr=dev(thr), want_sums=True)
    ctx.device_status()
    assert np.array_equal(sums.cpu().numpy(), S)
    got = bits.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, N), oracle.threshold(S, thr))
    assert padding_is_zero(got, N)
    ctx.set_workspace(None)
    del ws


def test_expand_signs_f4(ctx):
    x = wl.pm1(np.random.default_rng(4), (21, 300))
    p = ctx.pack_signs(dev(x, torch.int8))
    e = ctx.expand_signs_f4(p, 21, 300).cpu().numpy()
    assert e.shape == (21, 256)
    nib = np.stack([e & 0xF, e >> 4], axis=-1).reshape(21, -1)            # value k in byte k/2, even k low
    assert np.array_equal(nib[:, :300], np.where(x > 0, 0x2, 0xA)) and not nib[:, 300:].any()


def test_expand_signs(ctx):
    x = wl.pm1(np.random.default_rng(3), (37, 300))
    p = ctx.pack_signs(dev(x, torch.int8))
    e = ctx.expand_signs(p, 37, 300).cpu().numpy()
    assert e.shape == (37, 384) and np.array_equal(e[:, :300], x) and not e[:, 300:].any()


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("M,N,K", [(700, 520, 1000), (1030, 200, 4100), (300, 130, 64), (1, 1, 1), (1, 33, 31),
                                   (2, 1, 257), (129, 193, 300), (5, 400, 2), (257, 31, 513)])
def test_binary_dense_expanded(ctx, M, N, K, bits):
    """The tensor kernel on operands the caller keeps expanded: packed signs and the next layer's operand, chained
    through a second layer, against the oracle."""
    rng = np.random.default_rng(M + N + K + bits)
    A, W1, W2 = wl.pm1(rng, (M, K)), wl.pm1(rng, (N, K)), wl.pm1(rng, (96, N))
    thr1 = rng.integers(-30, 31, N).astype(np.int32)
    thr2 = rng.integers(-10, 11, 96).astype(np.int32)
    flip1 = rng.integers(0, 2, N).astype(np.uint8)
    h = oracle.threshold(oracle.gemm(A, W1.T.copy()), thr1, flip1)
    want2 = oracle.threshold(oracle.gemm(h, W2.T.copy()), thr2, np.zeros(96, np.uint8))
    expand = ctx.expand_signs_f4 if bits == 4 else ctx.expand_signs
    Ae = expand(ctx.pack_signs(dev(A, torch.int8)), M, K)
    W1e = expand(ctx.pack_signs(dev(W1, torch.int8)), N, K)
    W2e = expand(ctx.pack_signs(dev(W2, torch.int8)), 96, N)
    flip_p = dev(np_pack_pm1(2 * flip1.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    out, out_exp = ctx.binary_dense_expanded(Ae, W1e, bits, dev(thr1), flip_p, M, N, K, want_bits=True, want_exp=True)
    out2, _ = ctx.binary_dense_expanded(out_exp, W2e, bits, dev(thr2), None, M, 96, N)
    ctx.device_status()
    got = out.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, N), h) and padding_is_zero(got, N)
    # the expanded output equals the expansion of the packed one up to the end of the last 32-value group
    nb = (N + 31) // 32 * 32 // (2 if bits == 4 else 1)
    assert torch.equal(expand(out, M, N)[:, :nb].cpu().view(torch.uint8), out_exp[:, :nb].cpu().view(torch.uint8))
    assert np.array_equal(np_unpack_pm1(out2.cpu().numpy(), 96), want2)


@pytest.mark.parametrize("pre_expanded", [True, False])
@pytest.mark.parametrize("host_io", [False, True])
def test_mlp_forward_tensor_engine(ctx, host_io, pre_expanded):
    batch, sizes = 2000, (784, 1024, 1100, 1024, 10)
    case = wl.mlp_case(batch=batch, sizes=sizes, seed=77)
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"], expand_weights=pre_expanded)
    ws = with_ws(ctx, ctx.mlp_workspace_bytes(net["desc"], batch, host_io))
    if host_io:
        Xh = torch.from_numpy(case["X"]).pin_memory()
        Sh = torch.empty(batch, sizes[-1], dtype=torch.float32).pin_memory()
        ctx.mlp_forward_host(net["desc"], Xh, batch, Sh)
        ctx.device_status()
        got = Sh.numpy().astype(np.float64)
    else:
        hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
        scores = ctx.mlp_forward(net["desc"], dev(case["X"]), batch, hidden_out=hidden)
        ctx.device_status()
        for k, (g, w) in enumerate(zip(hidden, want_hidden)):
            gh = g.cpu().numpy()
            assert np.array_equal(np_unpack_pm1(gh, w.shape[1]), w), f"hidden layer {k}"
            assert padding_is_zero(gh, w.shape[1])
        got = scores.cpu().numpy().astype(np.float64)
    tol = 1e-5 * np.abs(want_scores) + 1e-6 * np.abs(want_scores).max()
    assert (np.abs(got - want_scores) <= tol).all()
    ctx.set_workspace(None)
    del ws


@pytest.mark.parametrize("B,H,W,Cin,Cout,pool", [(8, 32, 32, 128, 128, False), (8, 32, 32, 128, 200, True),
                                                 (16, 16, 16, 256, 256, True), (33, 8, 8, 512, 512, True),
                                                 (35, 8, 8, 256, 300, False), (3, 64, 64, 128, 128, True),
                                                 (300, 4, 4, 256, 128, True), (260, 4, 4, 128, 256, False),
                                                 (5, 16, 16, 512, 200, False), (9, 32, 32, 128, 384, False)])
@pytest.mark.parametrize("form", [0, 1], ids=["halo-tiles", "box-per-tap"])
def test_binary_conv2d_tensor_engine(ctx, B, H, W, Cin, Cout, pool, form):
    """Both ways the tensor engine brings a convolution's input into shared memory (bnn_set_conv_form): halo tiles (one slab
    per horizontal tap, read at three row offsets; several small images per tile are kept in (row, image, column) order)
    and one operand box per tap.  Image sizes 64, 32, 16, 8 and 4: one, one, one, two and eight images per 128-pixel tile."""
    ctx.set_conv_form(form)
    rng = np.random.default_rng(B + H + Cin + Cout)
    act = wl.pm1(rng, (B, H, W, Cin))
    wgt = wl.pm1(rng, (Cout, 3, 3, Cin))
    S = oracle.conv3x3(act, wgt)
    thr = rng.integers(-40, 41, Cout).astype(np.int32)
    thr[0] = S[0, 0, 0, 0]                       # a tie on a corner pixel (only 4 valid taps)
    flip = rng.integers(0, 2, Cout).astype(np.uint8)
    P = oracle.maxpool2x2(S) if pool else S
    want = oracle.threshold(P, thr, flip)
    actp = dev(np_pack_pm1(act).view(np.int32))
    Wp = dev(np_pack_pm1(wgt.reshape(Cout, 9, Cin)).reshape(Cout, -1).view(np.int32))
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    need = ctx.conv_workspace_bytes(B, H, W, Cin, Cout, pool)
    assert need > 0
    ws = with_ws(ctx, need)
    bits, sums = ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p, want_sums=not pool)
    ctx.device_status()
    if not pool:
        assert np.array_equal(sums.cpu().numpy(), S)
    got = bits.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, Cout), want)
    assert padding_is_zero(got, Cout)
    ctx.set_workspace(None)
    ctx.set_conv_form(0)
    del ws


@pytest.mark.parametrize("B,H,W,Cin,Cout,pool", [(20, 32, 32, 3, 128, False), (17, 32, 32, 3, 100, True), (70, 16, 16, 1, 64, True),
                                                 (300, 8, 8, 2, 300, False)])
def test_first_conv_u8_tensor_engine(ctx, B, H, W, Cin, Cout, pool):
    rng = np.random.default_rng(B + Cout)
    X = wl.u8(rng, (B, H, W, Cin))
    X[0] = 255
    wgt = wl.pm1(rng, (Cout, 3, 3, Cin))
    thr = rng.integers(-500, 500, Cout).astype(np.int32)
    flip = rng.integers(0, 2, Cout).astype(np.uint8)
    S = oracle.conv3x3(X, wgt)
    P = oracle.maxpool2x2(S) if pool else S
    Wp = dev(np_pack_pm1(wgt.reshape(Cout, 9 * Cin)).reshape(-1).view(np.int32))
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    need = ctx.conv_workspace_bytes(B, H, W, Cin, Cout, pool)
    assert need > 0
    ws = with_ws(ctx, need)
    bits, sums = ctx.binary_conv2d(dev(X), B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p, want_sums=not pool)
    ctx.device_status()
    if not pool:
        assert np.array_equal(sums.cpu().numpy(), S)
    got = bits.cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, Cout), oracle.threshold(P, thr, flip))
    assert padding_is_zero(got, Cout)
    ctx.set_workspace(None)
    del ws


def test_mlp_forward_unaligned_input_falls_back_cleanly(ctx):
    """An input whose rows are not 16-byte aligned cannot be fed to the tensor engine's TMA loads: the forward pass
    must run on the CUDA-core kernels without touching the activations it keeps in the same workspace."""
    batch, sizes = 2000, (790, 1024, 1024, 10)          # 790-byte rows: not a multiple of 16
    case = wl.mlp_case(batch=batch, sizes=sizes, seed=5)
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    ws = with_ws(ctx, ctx.mlp_workspace_bytes(net["desc"], batch, False))
    ctx.set_engine(binding.ENGINE_AUTO)
    hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
    scores = ctx.mlp_forward(net["desc"], dev(case["X"]), batch, hidden_out=hidden)
    ctx.device_status()
    ctx.set_engine(binding.ENGINE_TENSOR)
    for k, (g, w) in enumerate(zip(hidden, want_hidden)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[1]), w), f"hidden layer {k}"
    got = scores.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want_scores) <= 1e-5 * np.abs(want_scores) + 1e-6 * np.abs(want_scores).max()).all()
    ctx.set_workspace(None)
    del ws


@pytest.mark.parametrize("channels,hw,B", [((128, 128, 256, 128), 32, 20), ((128, 256, 256, 512, 256), 32, 20),
                                           ((128, 128, 256, 128), 16, 256), ((128, 128, 128, 128, 256, 256), 16, 256)])
@pytest.mark.parametrize("pre_expanded", [True, False])
def test_convnet_forward_chained_on_tensor_engine(ctx, pre_expanded, channels, hw, B):
    """bnn_convnet_forward with every layer on the tensor engine: +-1 values handed from layer to layer (pooled and not)
    as 4-bit nibbles: into layers with a multiple of 256 input channels (the second list has three of those in a row: not
    pooled, pooled, not pooled) and into layers with 128 (half-width K steps, rows of 64 bytes; the third list has them at
    every image size down to 4 x 4, where one tile holds several images).  The batches keep every layer above the sizes
    from which the engine takes it."""
    case = wl.convnet_case(batch=B, hw=hw, channels=channels, seed=9)
    want = oracle.convnet_forward(case["X"], case["layers"])
    net = nets.prepare_convnet(ctx, case["layers"], expand_weights=pre_expanded)
    desc, keep = ctx.make_convnet_desc(net)
    need = ctx.convnet_workspace_bytes(desc, B, hw, hw)
    ws = with_ws(ctx, need)
    outs = [torch.empty(w.shape[0], w.shape[1], w.shape[2], binding.words(w.shape[3]), dtype=torch.int32, device="cuda")
            for w in want]
    final = torch.empty_like(outs[-1])
    ctx.convnet_forward(desc, dev(case["X"]), B, hw, hw, final, layer_out=outs)
    ctx.device_status()
    for k, (g, w) in enumerate(zip(outs, want)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[-1]), w), f"conv layer {k}"
    assert torch.equal(final, outs[-1])
    ctx.set_workspace(None)
    del ws


def test_mlp_forward_host_on_a_side_stream_in_chunks():
    """Host-buffer forward large enough to be copied in two chunks (internal copy stream, events), on a context bound to
    a stream of its own, called twice back to back with different inputs and no synchronisation in between."""
    batch, sizes = 6400, (784, 1024, 1024, 10)
    cases = [wl.mlp_case(batch=batch, sizes=sizes, seed=s) for s in (31, 32)]
    cases[1]["weights"], cases[1]["bns"] = cases[0]["weights"], cases[0]["bns"]      # same network, other inputs
    wants = [oracle.mlp_forward(c["X"], c["weights"], c["bns"])[0] for c in cases]
    build.build()
    s = torch.cuda.Stream()
    c2 = binding.Context(0, stream=s)
    with torch.cuda.stream(s):
        net = nets.prepare_mlp(c2, cases[0]["weights"], cases[0]["bns"])
        ws = with_ws(c2, c2.mlp_workspace_bytes(net["desc"], batch, True))
        Xh = [torch.from_numpy(c["X"]).pin_memory() for c in cases]
        Sh = [torch.empty(batch, sizes[-1], dtype=torch.float32).pin_memory() for _ in cases]
        for x, o in zip(Xh, Sh):
            c2.mlp_forward_host(net["desc"], x, batch, o)
        c2.device_status()
    for o, want in zip(Sh, wants):
        got = o.numpy().astype(np.float64)
        assert (np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-6 * np.abs(want).max()).all()
    c2.set_workspace(None)
    c2.close()
    del ws


def test_back_to_back_calls_without_synchronisation(ctx):
    """Dependent launches let a kernel be set up while its predecessor still runs.  Many calls queued without a host
    synchronisation, alternating inputs and sharing one workspace (every call's expansion pass overwrites what the
    previous call's kernel read), must still give each call its own result."""
    M, N, K = 1500, 640, 2048
    rng = np.random.default_rng(123)
    As = [wl.pm1(rng, (M, K)) for _ in range(3)]
    W = wl.pm1(rng, (N, K))
    thr = rng.integers(-20, 21, N).astype(np.int32)
    wants = [oracle.threshold(oracle.gemm(A, W.T.copy()), thr) for A in As]
    Aps = [ctx.pack_signs(dev(A, torch.int8)) for A in As]
    Wp = ctx.pack_signs(dev(W, torch.int8))
    thr_d = dev(thr)
    ws = with_ws(ctx, ctx.gemm_workspace_bytes(M, N, K))
    outs = []
    for i in range(24):
        outs.append((i % 3, ctx.binary_dense(Aps[i % 3], Wp, thr_d, None, M, N, K)))
    # the whole MLP, alternating two batches, into separate score buffers
    batch, sizes = 2000, (784, 1024, 1100, 1024, 10)     # every hidden layer large enough for the tensor engine
    case = wl.mlp_case(batch=batch, sizes=sizes, seed=5)
    X2 = wl.u8(np.random.default_rng(6), (batch, sizes[0]))
    want_s = [oracle.mlp_forward(X, case["weights"], case["bns"])[0] for X in (case["X"], X2)]
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    ws2 = with_ws(ctx, ctx.mlp_workspace_bytes(net["desc"], batch, False))
    Xd = [dev(case["X"]), dev(X2)]
    scores = [(i % 2, ctx.mlp_forward(net["desc"], Xd[i % 2], batch)) for i in range(16)]
    ctx.device_status()
    for k, o in outs:
        assert np.array_equal(np_unpack_pm1(o.cpu().numpy(), N), wants[k])
    for k, sc in scores:
        got = sc.cpu().numpy().astype(np.float64)
        tol = 1e-5 * np.abs(want_s[k]) + 1e-6 * np.abs(want_s[k]).max()
        assert (np.abs(got - want_s[k]) <= tol).all()
    ctx.set_workspace(None)
    del ws, ws2


def test_last_tensor_kernel_clock_reports_a_plausible_sm_clock(ctx):
    """The kernel's own record of the SM clock it ran at (cycle counter against the nanosecond timer in its first CTA)."""
    M, N, K = 4096, 4096, 4096
    A, B = wl.gemm_case(M, N, K, seed=5)
    Ap = ctx.pack_signs(dev(A))
    Bp = ctx.pack_signs(dev(B), pack_along=1)
    ws = with_ws(ctx, ctx.gemm_workspace_bytes(M, N, K))
    C = torch.empty(M, N, dtype=torch.int32, device="cuda")
    for _ in range(3):
        ctx.xnor_gemm(Ap, Bp, M, N, K, C=C)
    mhz, us = ctx.last_tensor_kernel_clock()
    assert 300.0 < mhz < 2300.0, mhz
    assert 1.0 < us < 1000.0, us
    ctx.set_workspace(None)
    del ws
