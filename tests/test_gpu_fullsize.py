"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py
times (library-default inner loop).  Where the oracle cannot finish the whole problem in seconds it checks
sampled rows (first, last, tile-boundary and random ones) over all columns, and the complete output is
compared on the GPU with torch.matmul / conv2d of the +-1 values (exact: every partial sum is an integer
below 2^24)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, nets, workloads as wl
from util import np_unpack_pm1, padding_is_zero

pytestmark = pytest.mark.gpu
torch.backends.cuda.matmul.allow_tf32 = False
torch.backends.cudnn.allow_tf32 = False


@pytest.fixture(scope="module", params=[binding.ENGINE_POPC, binding.ENGINE_AUTO], ids=["popc", "auto"])
def ctx(request):
    """Both engines bench.py can time: the CUDA-core XOR-popcount kernels, and "auto" (the tensor-core int8
    engine wherever the shape qualifies and a workspace is set)."""
    build.build()
    c = binding.Context(0)
    c.set_engine(request.param)
    yield c
    torch.cuda.synchronize()
    c.close()


def give_gemm_workspace(ctx, M, N, K):
    ws = torch.empty(max(ctx.gemm_workspace_bytes(M, N, K), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    return ws


def sample_rows(M, n_random, rng):
    fixed = [0, 1, M - 1, M - 2]
    for t in (63, 64, 127, 128, 255, 256, M // 2 - 1, M // 2, M - 128, M - 129):
        if 0 <= t < M:
            fixed.append(t)
    rows = np.unique(np.concatenate([np.array(fixed), rng.integers(0, M, n_random)]))
    return rows[(rows >= 0) & (rows < M)]


def unpack_bits_gpu(words: torch.Tensor, n: int) -> torch.Tensor:
    """Packed int32 [R, ld] -> bool [R, n] on the GPU (test-side decoding of the ABI's bit layout)."""
    sh = torch.arange(32, device=words.device, dtype=torch.int32)
    bits = (words.unsqueeze(-1) >> sh) & 1
    return bits.reshape(words.shape[0], -1)[:, :n].bool()


@pytest.mark.parametrize("M,N,K", wl.GEMM_SWEEP)
def test_gemm_sweep_full_size(ctx, M, N, K):
    A, B = wl.gemm_case(M, N, K, seed=2)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    Ap = ctx.pack_signs(Ad)
    Bp = ctx.pack_signs(Bd, pack_along=1)
    assert Ap.shape[1] % 4 == 0 and Ap.shape[1] >= (K + 31) // 32
    if K % 32:   # "padded bits must not count": fill the padding of both operands with ones
        Ap[:, K // 32] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")
        Bp[:, K // 32] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")
        Ap[:, K // 32 + 1:] = -1
        Bp[:, K // 32 + 1:] = -1
    ws = give_gemm_workspace(ctx, M, N, K)
    C = ctx.xnor_gemm(Ap, Bp, M, N, K)
    ctx.device_status()
    # (a) complete output against the library matmul of the +-1 values, on the GPU
    ref = torch.matmul(Ad.float(), Bd.float())          # fp32, TF32 off: exact
    assert torch.equal(C.float(), ref)
    del ref
    # (b) sampled rows against the oracle
    rows = sample_rows(M, 48, np.random.default_rng(K))
    want = oracle.gemm(A[rows], B)
    assert np.array_equal(C[torch.from_numpy(rows).cuda()].cpu().numpy(), want)
    # (c) invariants at any size: parity and bound
    assert bool(((C - K) % 2 == 0).all()) and int(C.abs().max()) <= K


def test_mlp_config_full_batch(ctx):
    case = wl.mlp_case()           # batch 10000, 784-4096-4096-4096-10, seed 1
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    batch, sizes = case["batch"], case["sizes"]
    ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], batch, True), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
    scores = ctx.mlp_forward(net["desc"], torch.from_numpy(case["X"]).cuda(), batch, hidden_out=hidden)
    ctx.device_status()
    for k, (g, w) in enumerate(zip(hidden, want_hidden)):
        gh = g.cpu().numpy()
        assert np.array_equal(np_unpack_pm1(gh, w.shape[1]), w), f"hidden layer {k}"
        assert padding_is_zero(gh, w.shape[1])
    got = scores.cpu().numpy().astype(np.float64)
    tol = 1e-5 * np.abs(want_scores) + 1e-6 * np.abs(want_scores).max()
    assert (np.abs(got - want_scores) <= tol).all()
    assert np.array_equal(got.argmax(1), want_scores.argmax(1))
    # the host-buffer entry point gives the same scores
    Xh = torch.from_numpy(case["X"]).pin_memory()
    Sh = torch.empty(batch, sizes[-1], dtype=torch.float32).pin_memory()
    ctx.mlp_forward_host(net["desc"], Xh, batch, Sh)
    torch.cuda.synchronize()
    assert np.array_equal(Sh.numpy(), scores.cpu().numpy())
    ctx.set_workspace(None)


def test_convnet_config_full_batch(ctx):
    case = wl.convnet_case()       # batch 256, 32x32x3, 128-128-256-256-512-512, seed 3
    net = nets.prepare_convnet(ctx, case["layers"])
    Xd = torch.from_numpy(case["X"]).cuda()
    ws = torch.empty(max(nets.convnet_workspace_bytes(ctx, net, case["batch"], case["hw"], case["hw"]), 256),
                     dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    outs = nets.convnet_forward(ctx, net, Xd, keep_all=True)
    ctx.device_status()
    # (a) oracle, every layer, on the first and last images of the batch
    pick = np.r_[0:12, 244:256]
    want = oracle.convnet_forward(case["X"][pick], case["layers"])
    for k, (g, w) in enumerate(zip(outs, want)):
        gh = g[torch.from_numpy(pick).cuda()].cpu().numpy()
        assert np.array_equal(np_unpack_pm1(gh, w.shape[-1]), w), f"conv layer {k}"
    # the whole-network entry point gives the same maps as the per-layer calls
    desc, keep = ctx.make_convnet_desc(net)
    ws2 = torch.empty(max(ctx.convnet_workspace_bytes(desc, case["batch"], case["hw"], case["hw"]), 256), dtype=torch.uint8,
                      device="cuda")
    ctx.set_workspace(ws2)
    outs2 = [torch.empty_like(o) for o in outs]
    final = torch.empty_like(outs[-1])
    ctx.convnet_forward(desc, Xd, case["batch"], case["hw"], case["hw"], final, layer_out=outs2)
    ctx.device_status()
    for k, (a1, a2) in enumerate(zip(outs, outs2)):
        assert torch.equal(a1, a2), f"bnn_convnet_forward layer {k}"
    assert torch.equal(final, outs[-1])
    # (b) every image, layer by layer, against torch conv2d on the GPU fed with the library's own previous layer
    B = case["batch"]
    a = Xd.float().permute(0, 3, 1, 2)
    for k, (L, P) in enumerate(zip(case["layers"], net)):
        w = torch.from_numpy(L["wgt"]).cuda().float().permute(0, 3, 1, 2)
        s = torch.round(torch.nn.functional.conv2d(a, w, padding=1))   # integers; cuDNN may pick a transform-based algorithm
        if L["pool"]:
            s = torch.nn.functional.max_pool2d(s, 2)
        s = s.permute(0, 2, 3, 1).contiguous()                       # B, H, W, Cout  (exact integers in fp32)
        Cout = s.shape[-1]
        thr = P["thr"].float()
        flipw = P["flip"]
        flip = unpack_bits_gpu(flipw.reshape(1, -1), Cout)[0]
        want_bits = (s >= thr) ^ flip
        got_bits = unpack_bits_gpu(outs[k].reshape(-1, outs[k].shape[-1]), Cout).reshape(want_bits.shape)
        assert torch.equal(got_bits, want_bits), f"conv layer {k} (all {B} images)"
        a = (got_bits.float() * 2 - 1).permute(0, 3, 1, 2)


@pytest.mark.parametrize("batch", wl.DENSE_BATCHES)
def test_dense_batch_sweep(ctx, batch):
    case = wl.dense_case(batch)
    K = N = 4096
    Ad, Wd = torch.from_numpy(case["A"]).cuda(), torch.from_numpy(case["W"]).cuda()
    Ap = ctx.pack_signs(Ad)
    Wp = ctx.pack_signs(Wd, pack_along=1)
    thr = torch.from_numpy(case["thr"]).cuda()
    ws = give_gemm_workspace(ctx, batch, N, K)
    out = ctx.binary_dense(Ap, Wp, thr, None, batch, N, K)
    ctx.device_status()
    # complete output against the library matmul on the GPU
    ref = torch.matmul(Ad.float(), Wd.float())          # fp32, TF32 off: exact
    assert torch.equal(unpack_bits_gpu(out, N), ref >= thr.float())
    # oracle on (sampled) rows
    rows = np.arange(batch) if batch <= 4096 else sample_rows(batch, 1000, np.random.default_rng(batch))
    want = oracle.threshold(oracle.gemm(case["A"][rows], case["W"]), case["thr"])
    got = out[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert np.array_equal(np_unpack_pm1(got, N), want)
    assert padding_is_zero(got, N)


# ------------------------------------------------------------------ the paper's other network shapes (layer lists are data)
def test_mlp_2048_unit_variant(ctx):
    """Section 2.2: the Torch7 MNIST MLP uses 2048-unit hidden layers; same kernels, another layer list."""
    case = wl.mlp_case(batch=4000, sizes=(784, 2048, 2048, 2048, 10), seed=6)
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    batch, sizes = case["batch"], case["sizes"]
    ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], batch, False), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
    scores = ctx.mlp_forward(net["desc"], torch.from_numpy(case["X"]).cuda(), batch, hidden_out=hidden)
    ctx.device_status()
    for k, (g, w) in enumerate(zip(hidden, want_hidden)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[1]), w), f"hidden layer {k}"
    got = scores.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want_scores) <= 1e-5 * np.abs(want_scores) + 1e-6 * np.abs(want_scores).max()).all()
    ctx.set_workspace(None)


def test_convnet_half_width_variant_with_dense_tail(ctx):
    """Section 2.4: the SVHN ConvNet has half the feature maps (64-64-128-128-256-256).  A fully-connected binary tail
    (flattened 4 x 4 x 256 map -> 1024 -> 10-way scores) is added with the dense-layer calls: the packed NHWC map of
    one image is already a packed row of 4096 bits."""
    B = 40
    case = wl.convnet_case(batch=B, channels=(64, 64, 128, 128, 256, 256), seed=11)
    want_maps = oracle.convnet_forward(case["X"], case["layers"])
    net = nets.prepare_convnet(ctx, case["layers"])
    desc, keep = ctx.make_convnet_desc(net)
    ws = torch.empty(max(ctx.convnet_workspace_bytes(desc, B, 32, 32), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    outs = [torch.empty(w.shape[0], w.shape[1], w.shape[2], binding.words(w.shape[3]), dtype=torch.int32, device="cuda")
            for w in want_maps]
    final = torch.empty_like(outs[-1])
    ctx.convnet_forward(desc, torch.from_numpy(case["X"]).cuda(), B, 32, 32, final, layer_out=outs)
    ctx.device_status()
    for k, (g, w) in enumerate(zip(outs, want_maps)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[-1]), w), f"conv layer {k}"
    # dense tail on the flattened map
    rng = np.random.default_rng(12)
    K = 4 * 4 * 256
    W1, W2 = wl.pm1(rng, (K, 1024)), wl.pm1(rng, (1024, 10))
    bn1, bn2 = wl.batchnorm_params(rng, 1024, K), wl.batchnorm_params(rng, 10, 1024)
    flat = want_maps[-1].reshape(B, K)                                  # NHWC flattening = (y, x, c) order
    h1 = oracle.sign_batchnorm(oracle.gemm(flat, W1), bn1)
    want_scores = oracle.batchnorm(oracle.gemm(h1, W2), bn2)
    thr1, flip1 = nets.fold(ctx, bn1, K)
    W1p, W2p = nets.pack_weight(ctx, W1), nets.pack_weight(ctx, W2)
    ctx.set_workspace(None)
    a1 = ctx.binary_dense(final.reshape(B, K // 32), W1p, thr1, flip1, B, 1024, K)
    S = ctx.xnor_gemm(a1, W2p, B, 10, 1024)
    ctx.device_status()
    assert np.array_equal(np_unpack_pm1(a1.cpu().numpy(), 1024), h1)
    got = oracle.batchnorm(S.cpu().numpy(), bn2)                        # integer sums from the GPU, float epilogue on the host
    assert np.array_equal(S.cpu().numpy(), oracle.gemm(h1, W2))
    assert np.allclose(got, want_scores, rtol=0, atol=0)


# ------------------------------------------------------------------ the other literal readings of the two network configurations
def test_mlp_other_reading_four_wide_layers(ctx):
    """The MLP configuration can also be read as "a first layer, THEN three more binary layers of 4096 units": weights
    784x4096, three times 4096x4096, 4096x10 (one 4096x4096 layer more than the paper's topology, Section 2.1).  The layer
    list is data: same calls, every hidden layer against the oracle."""
    case = wl.mlp_case(batch=2500, sizes=(784, 4096, 4096, 4096, 4096, 10), seed=21)
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    batch, sizes = case["batch"], case["sizes"]
    ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], batch, False), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
    scores = ctx.mlp_forward(net["desc"], torch.from_numpy(case["X"]).cuda(), batch, hidden_out=hidden)
    ctx.device_status()
    assert len(hidden) == 4
    for k, (g, w) in enumerate(zip(hidden, want_hidden)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[1]), w), f"hidden layer {k}"
    got = scores.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want_scores) <= 1e-5 * np.abs(want_scores) + 1e-6 * np.abs(want_scores).max()).all()
    assert np.array_equal(got.argmax(1), want_scores.argmax(1))
    ctx.set_workspace(None)


def other_reading_convnet(batch, seed=22):
    """The ConvNet configuration read as "a first layer, THEN binary convolutions of widths 128-128-256-256-512-512":
    seven convolutions, the 8-bit one followed by six binary ones (one 128 -> 128 convolution more than the paper's
    topology), a 2x2 max-pool after every second binary one."""
    case = wl.convnet_case(batch=batch, channels=(128, 128, 128, 256, 256, 512, 512), seed=seed)
    for i, L in enumerate(case["layers"]):
        L["pool"] = i in (2, 4, 6)
    return case


def test_convnet_other_reading_seven_convolutions(ctx):
    B = 16
    case = other_reading_convnet(B)
    want_maps = oracle.convnet_forward(case["X"], case["layers"])
    assert want_maps[-1].shape == (B, 4, 4, 512)
    net = nets.prepare_convnet(ctx, case["layers"])
    desc, keep = ctx.make_convnet_desc(net)
    ws = torch.empty(max(ctx.convnet_workspace_bytes(desc, B, 32, 32), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    outs = [torch.empty(w.shape[0], w.shape[1], w.shape[2], binding.words(w.shape[3]), dtype=torch.int32, device="cuda")
            for w in want_maps]
    final = torch.empty_like(outs[-1])
    ctx.convnet_forward(desc, torch.from_numpy(case["X"]).cuda(), B, 32, 32, final, layer_out=outs)
    ctx.device_status()
    for k, (g, w) in enumerate(zip(outs, want_maps)):
        assert np.array_equal(np_unpack_pm1(g.cpu().numpy(), w.shape[-1]), w), f"conv layer {k}"
    assert torch.equal(final, outs[-1])
    ctx.set_workspace(None)


def test_full_width_convnet_with_dense_tail(ctx):
    """Sections 2.3-2.4: the CIFAR-10 ConvNet ends in fully-connected binary layers.  The full-width convolution stack
    (128-128-256-256-512-512) followed by 8192 -> 1024 -> 1024 -> 10 on the flattened 4 x 4 x 512 map: the packed NHWC map
    of one image is already a packed row of 8192 bits, so the tail is two fused dense calls and one plain product."""
    B = 24
    case = wl.convnet_case(batch=B, seed=23)
    want_maps = oracle.convnet_forward(case["X"], case["layers"])
    net = nets.prepare_convnet(ctx, case["layers"])
    desc, keep = ctx.make_convnet_desc(net)
    ws = torch.empty(max(ctx.convnet_workspace_bytes(desc, B, 32, 32), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    final = torch.empty(B, 4, 4, 16, dtype=torch.int32, device="cuda")
    ctx.convnet_forward(desc, torch.from_numpy(case["X"]).cuda(), B, 32, 32, final)
    ctx.device_status()
    assert np.array_equal(np_unpack_pm1(final.cpu().numpy(), 512), want_maps[-1])
    rng = np.random.default_rng(24)
    K = 4 * 4 * 512
    W1, W2, W3 = wl.pm1(rng, (K, 1024)), wl.pm1(rng, (1024, 1024)), wl.pm1(rng, (1024, 10))
    bn1, bn2, bn3 = wl.batchnorm_params(rng, 1024, K), wl.batchnorm_params(rng, 1024, 1024), wl.batchnorm_params(rng, 10, 1024)
    flat = want_maps[-1].reshape(B, K)                                  # NHWC flattening = (y, x, c) order
    h1 = oracle.sign_batchnorm(oracle.gemm(flat, W1), bn1)
    h2 = oracle.sign_batchnorm(oracle.gemm(h1, W2), bn2)
    want_sums = oracle.gemm(h2, W3)
    thr1, flip1 = nets.fold(ctx, bn1, K)
    thr2, flip2 = nets.fold(ctx, bn2, 1024)
    W1p, W2p, W3p = (nets.pack_weight(ctx, W) for W in (W1, W2, W3))
    ctx.set_workspace(None)
    a1 = ctx.binary_dense(final.reshape(B, K // 32), W1p, thr1, flip1, B, 1024, K)
    a2 = ctx.binary_dense(a1, W2p, thr2, flip2, B, 1024, 1024)
    S = ctx.xnor_gemm(a2, W3p, B, 10, 1024)
    ctx.device_status()
    assert np.array_equal(np_unpack_pm1(a1.cpu().numpy(), 1024), h1)
    assert np.array_equal(np_unpack_pm1(a2.cpu().numpy(), 1024), h2)
    assert np.array_equal(S.cpu().numpy(), want_sums)
    got = oracle.batchnorm(S.cpu().numpy(), bn3)                        # integer sums from the GPU; the affine is the oracle's
    assert np.array_equal(got.argmax(1), oracle.batchnorm(want_sums, bn3).argmax(1))
