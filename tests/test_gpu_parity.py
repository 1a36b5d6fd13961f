"""GPU parity: every C-ABI call against the CPU oracle, element by element, bit-exact for all integer,
sign and packed outputs; the float scores of the output layer to 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, nets, workloads as wl
from util import np_pack_pm1, np_unpack_pm1, padding_is_zero

pytestmark = pytest.mark.gpu

VARIANTS = [binding.VARIANT_PLAIN, binding.VARIANT_CSA]


@pytest.fixture(scope="module", params=[16, 8], ids=["rows16", "rows8"])
def ctx(request):
    """The CUDA-core kernels in both register-tile shapes (no workspace is set, so nothing goes to the tensor engine)."""
    build.build()
    c = binding.Context(0)
    c.set_tile_rows(request.param)
    yield c
    torch.cuda.synchronize()
    c.close()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t if dtype is None else t.to(dtype)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


# ------------------------------------------------------------------ bnn_pack_signs
@pytest.mark.parametrize("rows,cols", [(1, 1), (3, 31), (2, 32), (5, 33), (7, 100), (64, 512), (33, 4100), (130, 257)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.int8])
def test_pack_signs_along_cols(ctx, rows, cols, dtype):
    rng = np.random.default_rng(rows * 1000 + cols)
    if dtype == torch.int8:
        x = rng.integers(-128, 128, (rows, cols)).astype(np.int8)
    else:
        x = rng.normal(size=(rows, cols)).astype(np.float32)
        x[rng.random((rows, cols)) < 0.1] = 0.0
        x[rng.random((rows, cols)) < 0.05] = -0.0
    want = oracle.sign(x.astype(np.float32) if dtype != torch.int8 else x.astype(np.int32))
    got = host(ctx.pack_signs(dev(x, dtype)))
    assert got.shape == (rows, binding.packed_ld(cols))
    assert np.array_equal(np_unpack_pm1(got, cols), want)
    assert padding_is_zero(got, cols)
    assert np.array_equal(got.view(np.uint32), np_pack_pm1(want, binding.packed_ld(cols)))


@pytest.mark.parametrize("K,N", [(1, 1), (31, 3), (33, 65), (512, 256), (100, 40), (300, 33)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.int8])
def test_pack_signs_along_rows_transposes(ctx, K, N, dtype):
    rng = np.random.default_rng(K * 7 + N)
    x = wl.pm1(rng, (K, N))
    got = host(ctx.pack_signs(dev(x, dtype), pack_along=1))
    assert got.shape == (N, binding.packed_ld(K))
    assert np.array_equal(np_unpack_pm1(got, K), x.T)
    assert padding_is_zero(got, K)


def test_pack_signs_64bit_words_are_the_same_bytes(ctx):
    x = wl.pm1(np.random.default_rng(1), (9, 200))
    a = host(ctx.pack_signs(dev(x, torch.int8), word_bits=32))
    b = host(ctx.pack_signs(dev(x, torch.int8), word_bits=64))
    assert np.array_equal(a, b)
    w64 = np.ascontiguousarray(b).view(np.uint64)
    k = 70
    assert ((int(w64[0, k // 64]) >> (k % 64)) & 1) == (1 if x[0, k] > 0 else 0)


# ------------------------------------------------------------------ bnn_xnor_gemm
def gemm_gpu(ctx, A, B):
    M, K = A.shape
    N = B.shape[1]
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Bp = ctx.pack_signs(dev(B, torch.int8), pack_along=1)
    return host(ctx.xnor_gemm(Ap, Bp, M, N, K))


SMALL = [(1, 1, 1), (2, 3, 31), (3, 2, 32), (33, 1, 33), (1, 33, 63), (5, 7, 64), (4, 4, 65), (3, 5, 100),
         (33, 33, 100), (40, 130, 257), (64, 256, 512), (129, 127, 300), (200, 260, 1000), (257, 129, 4100),
         # many rows times few columns (the output layer as a plain product): small-operand kernel with the roles swapped
         (300, 10, 4096), (1000, 32, 100), (77, 17, 33)]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("M,N,K", SMALL)
def test_xnor_gemm_small_and_ragged(ctx, M, N, K, variant):
    ctx.set_popc_variant(variant)
    A, B = wl.gemm_case(M, N, K, seed=M * 31 + N * 7 + K)
    assert np.array_equal(gemm_gpu(ctx, A, B), oracle.gemm(A, B))
    ctx.set_popc_variant(0)


def test_xnor_gemm_config1(ctx):
    A, B = wl.config1()
    C = gemm_gpu(ctx, A, B)
    assert C.shape == (64, 256) and np.array_equal(C, oracle.gemm(A, B))


@pytest.mark.parametrize("variant", VARIANTS)
def test_xnor_gemm_several_tiles_ragged(ctx, variant):
    ctx.set_popc_variant(variant)
    for (M, N, K) in [(300, 500, 777), (1000, 700, 2100), (2500, 19000, 96)]:
        A, B = wl.gemm_case(M, N, K, seed=K)
        assert np.array_equal(gemm_gpu(ctx, A, B), oracle.gemm(A, B))
    ctx.set_popc_variant(0)


def test_xnor_gemm_ignores_garbage_in_padding(ctx):
    M, N, K = 70, 140, 4100 - 4000    # K = 100: 4 words, 28 pad bits, ld = 4
    A, B = wl.gemm_case(M, N, K, seed=9)
    Ap = ctx.pack_signs(dev(A, torch.int8), dst_ld_w=8)
    Bp = ctx.pack_signs(dev(B, torch.int8), pack_along=1, dst_ld_w=8)
    Ap[:, 3] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")   # set every pad bit
    Bp[:, 3] |= torch.tensor(-1 << (K % 32), dtype=torch.int32, device="cuda")
    Ap[:, 4:] = 0x5A5A5A5A
    Bp[:, 4:] = 0x13579BDF
    assert np.array_equal(host(ctx.xnor_gemm(Ap, Bp, M, N, K)), oracle.gemm(A, B))
    # the skinny path too
    assert np.array_equal(host(ctx.xnor_gemm(Ap[:5].contiguous(), Bp, 5, N, K)), oracle.gemm(A[:5], B))


def test_xnor_gemm_strided_output_and_guard_bands(ctx):
    M, N, K = 77, 150, 333
    A, B = wl.gemm_case(M, N, K, seed=3)
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Bp = ctx.pack_signs(dev(B, torch.int8), pack_along=1)
    ldc = N + 10
    big = torch.full((M + 2, ldc), 12345, dtype=torch.int32, device="cuda")
    ctx.xnor_gemm(Ap, Bp, M, N, K, C=big[1:], ldc=ldc)
    out = host(big)
    assert np.array_equal(out[1:M + 1, :N], oracle.gemm(A, B))
    assert (out[0] == 12345).all() and (out[M + 1] == 12345).all() and (out[:, N:] == 12345).all()


def test_zero_sizes_and_errors(ctx):
    A, B = wl.gemm_case(4, 4, 64, seed=1)
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Bp = ctx.pack_signs(dev(B, torch.int8), pack_along=1)
    C = torch.full((4, 4), 7, dtype=torch.int32, device="cuda")
    ctx.xnor_gemm(Ap, Bp, 0, 4, 64, C=C)
    ctx.xnor_gemm(Ap, Bp, 4, 0, 64, C=C)
    assert (host(C) == 7).all()
    ctx.xnor_gemm(Ap, Bp, 4, 4, 0, C=C)                      # empty sum
    assert (host(C) == 0).all()
    L = binding.lib()
    h = ctx._h
    p = lambda t: t.data_ptr()
    assert L.bnn_xnor_gemm(h, p(Ap), 4, p(Bp), 4, None, 4, 4, 4, 64) == -1          # NULL output
    assert L.bnn_xnor_gemm(h, p(Ap), 4, p(Bp), 4, p(C), 4, -1, 4, 64) == -1         # negative size
    assert L.bnn_xnor_gemm(h, p(Ap), 1, p(Bp), 4, p(C), 4, 4, 4, 64) == -1          # ld < words
    assert L.bnn_xnor_gemm(h, p(Ap), 6, p(Bp), 4, p(C), 4, 4, 4, 64) == -2          # ld % 4
    assert L.bnn_xnor_gemm(h, p(Ap) + 4, 4, p(Bp), 4, p(C), 4, 4, 4, 64) == -2      # misaligned base
    assert L.bnn_xnor_gemm(h, p(Ap), 4, p(Bp), 4, p(C), 2, 4, 4, 64) == -1          # ldc < N
    assert L.bnn_binary_dense(h, p(Ap), 4, p(Bp), 4, None, None, p(C), 4, 4, 4, 64) == -1   # thr missing
    assert L.bnn_pack_signs(h, p(Ap), 7, 4, 4, 4, 0, 32, p(C), 4) == -1             # unknown dtype
    assert L.bnn_pack_signs(h, p(Ap), 2, 4, 4, 4, 0, 48, p(C), 4) == -1             # word width
    torch.cuda.synchronize()


# ------------------------------------------------------------------ bnn_binary_dense
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("M,N,K,use_flip", [(1, 64, 128, False), (16, 96, 200, True), (33, 100, 77, True),
                                            (130, 257, 513, True), (300, 4096, 256, False), (260, 130, 4096, True)])
def test_binary_dense(ctx, M, N, K, use_flip, variant):
    ctx.set_popc_variant(variant)
    rng = np.random.default_rng(M + N + K)
    A, W = wl.gemm_case(M, N, K, seed=M + N + K)
    S = oracle.gemm(A, W)
    thr = rng.integers(-20, 21, N).astype(np.int32)
    thr[: min(N, M)] = S[np.arange(min(N, M)), np.arange(min(N, M))]    # exact ties on the diagonal
    thr[-1] = K + 1
    thr[-2 % N] = -K
    flip = rng.integers(0, 2, N).astype(np.uint8) if use_flip else None
    want = oracle.threshold(S, thr, flip)
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32)) if use_flip else None
    ld = binding.packed_ld(N) + 4
    out = torch.full((M, ld), -1, dtype=torch.int32, device="cuda")
    ctx.binary_dense(Ap, Wp, dev(thr), flip_p, M, N, K, out=out, ldo_w=ld)
    got = host(out)
    assert np.array_equal(np_unpack_pm1(got, N), want)
    assert padding_is_zero(got, N)
    ctx.set_popc_variant(0)


def test_binary_dense_extreme_thresholds(ctx):
    M, N, K = 40, 64, 96
    A, W = wl.gemm_case(M, N, K, seed=2)
    Ap = ctx.pack_signs(dev(A, torch.int8))
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    for t, val in [(2**31 - 1, -1), (-2**31, 1), (K + 1, -1), (-K, 1)]:
        thr = np.full(N, t, dtype=np.int64).astype(np.int32)
        got = np_unpack_pm1(host(ctx.binary_dense(Ap, Wp, dev(thr), None, M, N, K)), N)
        assert (got == val).all()


# ------------------------------------------------------------------ bnn_first_layer_bitplanes
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 31), (7, 33, 32), (40, 130, 100), (130, 64, 784), (300, 200, 50)])
def test_first_layer_bitplanes(ctx, M, N, K):
    rng = np.random.default_rng(M * 3 + N * 5 + K)
    X = wl.u8(rng, (M, K))
    X[0, :] = 255
    if M > 1:
        X[1, :] = 0
    W = wl.pm1(rng, (K, N))
    S = oracle.first_layer(X, W)
    thr = rng.integers(-3000, 3000, N).astype(np.int32)
    thr[0] = S[0, 0]
    flip = rng.integers(0, 2, N).astype(np.uint8)
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    bits, sums = ctx.first_layer_bitplanes(dev(X), Wp, M, N, K, thr=dev(thr), flip=flip_p, want_sums=True)
    assert np.array_equal(host(sums), S)
    got = host(bits)
    assert np.array_equal(np_unpack_pm1(got, N), oracle.threshold(S, thr, flip))
    assert padding_is_zero(got, N)


@pytest.mark.parametrize("M,N,K", [(70, 512, 784), (33, 600, 53), (260, 1024, 100), (9, 512, 1)])
def test_first_layer_with_presplit_planes(ctx, M, N, K):
    """With a workspace the CUDA-core first layer splits the bytes into bit-planes once, in a pre-pass."""
    rng = np.random.default_rng(M + N + K)
    X, W = wl.u8(rng, (M, K)), wl.pm1(rng, (K, N))
    X[0, :] = 255
    S = oracle.first_layer(X, W)
    thr = rng.integers(-2000, 2000, N).astype(np.int32)
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    ws = torch.empty(8 << 20, dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    ctx.set_engine(binding.ENGINE_POPC)
    bits, sums = ctx.first_layer_bitplanes(dev(X), Wp, M, N, K, thr=dev(thr), want_sums=True)
    ctx.set_engine(binding.ENGINE_AUTO)
    ctx.set_workspace(None)
    assert np.array_equal(host(sums), S)
    got = host(bits)
    assert np.array_equal(np_unpack_pm1(got, N), oracle.threshold(S, thr))
    assert padding_is_zero(got, N)


def test_first_layer_unaligned_rows(ctx):
    M, N, K = 20, 40, 53            # row stride 53 bytes: the 16-byte fast path must not be taken blindly
    rng = np.random.default_rng(0)
    X, W = wl.u8(rng, (M, K)), wl.pm1(rng, (K, N))
    Wp = ctx.pack_signs(dev(W, torch.int8), pack_along=1)
    _, sums = ctx.first_layer_bitplanes(dev(X), Wp, M, N, K, want_bits=False, want_sums=True)
    assert np.array_equal(host(sums), oracle.first_layer(X, W))


# ------------------------------------------------------------------ bnn_binary_conv2d
def conv_case(B, H, W, Cin, Cout, seed):
    rng = np.random.default_rng(seed)
    act = wl.pm1(rng, (B, H, W, Cin))
    wgt = wl.pm1(rng, (Cout, 3, 3, Cin))
    thr = rng.integers(-30, 31, Cout).astype(np.int32)
    flip = rng.integers(0, 2, Cout).astype(np.uint8)
    return act, wgt, thr, flip


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("B,H,W,Cin,Cout,pool", [(1, 1, 1, 32, 32, False), (2, 2, 2, 32, 40, True),
                                                 (2, 5, 7, 64, 33, False), (3, 8, 6, 128, 130, True),
                                                 (2, 8, 8, 128, 128, False), (5, 6, 10, 96, 64, True),
                                                 (1, 16, 16, 256, 256, True)])
def test_binary_conv2d(ctx, B, H, W, Cin, Cout, pool, variant):
    ctx.set_popc_variant(variant)
    act, wgt, thr, flip = conv_case(B, H, W, Cin, Cout, seed=H * W + Cin + Cout)
    S = oracle.conv3x3(act, wgt)
    if pool:
        S = oracle.maxpool2x2(S)
    want = oracle.threshold(S, thr, flip)
    actp = dev(np_pack_pm1(act).view(np.int32))
    Wp = dev(np_pack_pm1(wgt.reshape(Cout, 9, Cin)).reshape(Cout, -1).view(np.int32))
    flip_p = dev(np_pack_pm1(2 * flip.astype(np.int8)[None, :] - 1)[0].view(np.int32))
    bits, sums = ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), flip=flip_p, want_sums=True)
    assert np.array_equal(host(sums), S)
    got = host(bits)
    assert np.array_equal(np_unpack_pm1(got, Cout), want)
    assert padding_is_zero(got, Cout)
    ctx.set_popc_variant(0)


@pytest.mark.parametrize("B,H,W,Cin,Cout,pool", [(2, 6, 6, 3, 128, False), (1, 4, 4, 3, 40, True), (2, 5, 3, 1, 7, False)])
def test_first_conv_u8_bitplanes(ctx, B, H, W, Cin, Cout, pool):
    rng = np.random.default_rng(B + H + Cout)
    X = wl.u8(rng, (B, H, W, Cin))
    wgt = wl.pm1(rng, (Cout, 3, 3, Cin))
    thr = rng.integers(-500, 500, Cout).astype(np.int32)
    S = oracle.conv3x3(X, wgt)
    if pool:
        S = oracle.maxpool2x2(S)
    Wp = dev(np_pack_pm1(wgt.reshape(Cout, 9 * Cin)).reshape(-1).view(np.int32))
    bits, sums = ctx.binary_conv2d(dev(X), B, H, W, Cin, Wp, Cout, pool=pool, thr=dev(thr), want_sums=True)
    assert np.array_equal(host(sums), S)
    assert np.array_equal(np_unpack_pm1(host(bits), Cout), oracle.threshold(S, thr))


def test_convnet_small_layer_by_layer(ctx):
    case = wl.convnet_case(batch=3, hw=8, channels=(128, 128, 256, 256), seed=3)
    want = oracle.convnet_forward(case["X"], case["layers"])
    net = nets.prepare_convnet(ctx, case["layers"])
    outs = nets.convnet_forward(ctx, net, dev(case["X"]), keep_all=True)
    for k, (g, w) in enumerate(zip(outs, want)):
        assert np.array_equal(np_unpack_pm1(host(g), w.shape[-1]), w), f"conv layer {k}"


def test_convnet_forward_call_layer_by_layer(ctx):
    """bnn_convnet_forward on the CUDA-core kernels (shapes too small for the tensor engine): every layer's map."""
    case = wl.convnet_case(batch=3, hw=8, channels=(128, 96, 256, 64), seed=4)
    want = oracle.convnet_forward(case["X"], case["layers"])
    net = nets.prepare_convnet(ctx, case["layers"], expand_weights=False)
    desc, keep = ctx.make_convnet_desc(net)
    ws = torch.empty(max(ctx.convnet_workspace_bytes(desc, 3, 8, 8), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    outs = [torch.empty(w.shape[0], w.shape[1], w.shape[2], binding.words(w.shape[3]), dtype=torch.int32, device="cuda")
            for w in want]
    final = torch.empty_like(outs[-1])
    ctx.convnet_forward(desc, dev(case["X"]), 3, 8, 8, final, layer_out=outs)
    for k, (g, w) in enumerate(zip(outs, want)):
        assert np.array_equal(np_unpack_pm1(host(g), w.shape[-1]), w), f"conv layer {k}"
    assert np.array_equal(host(final), host(outs[-1]))
    ctx.set_workspace(None)
    with pytest.raises(binding.BnnError) as e:
        ctx.convnet_forward(desc, dev(case["X"]), 3, 8, 8, final)
    assert e.value.status == -3


# ------------------------------------------------------------------ bnn_mlp_forward
def run_mlp(ctx, case, host_io=False):
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    batch = case["batch"]
    ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], batch, host_io), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    sizes = case["sizes"]
    if host_io:
        Xh = torch.from_numpy(case["X"]).pin_memory()
        Sh = torch.empty(batch, sizes[-1], dtype=torch.float32).pin_memory()
        ctx.mlp_forward_host(net["desc"], Xh, batch, Sh)
        torch.cuda.synchronize()
        ctx.set_workspace(None)
        return Sh.numpy().copy(), None
    hidden = [torch.empty(batch, binding.packed_ld(n), dtype=torch.int32, device="cuda") for n in sizes[1:-1]]
    scores = ctx.mlp_forward(net["desc"], dev(case["X"]), batch, hidden_out=hidden)
    out = host(scores), [host(h) for h in hidden]
    ctx.set_workspace(None)
    return out


def check_scores(got, want):
    # relative 1e-5 with an absolute floor for values that are (nearly) exact zeros
    tol = 1e-5 * np.abs(want) + 1e-6 * np.abs(want).max()
    assert (np.abs(got.astype(np.float64) - want) <= tol).all()
    assert np.array_equal(got.argmax(1), want.argmax(1))


@pytest.mark.parametrize("batch,sizes", [(1, (784, 256, 128, 10)), (37, (50, 64, 40, 10)), (300, (784, 512, 256, 256, 10)),
                                         (130, (100, 4096, 4096, 10))])
def test_mlp_forward_layer_by_layer(ctx, batch, sizes):
    case = wl.mlp_case(batch=batch, sizes=sizes, seed=batch)
    want_scores, want_hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    scores, hidden = run_mlp(ctx, case)
    for k, (g, w) in enumerate(zip(hidden, want_hidden)):
        assert np.array_equal(np_unpack_pm1(g, w.shape[1]), w), f"hidden layer {k}"
        assert padding_is_zero(g, w.shape[1])
    check_scores(scores, want_scores)


def test_mlp_forward_host_buffers(ctx):
    case = wl.mlp_case(batch=200, sizes=(784, 512, 512, 10), seed=8)
    want_scores, _ = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    scores, _ = run_mlp(ctx, case, host_io=True)
    check_scores(scores, want_scores)


def test_mlp_forward_needs_workspace(ctx):
    case = wl.mlp_case(batch=4, sizes=(32, 32, 10), seed=1)
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    ctx.set_workspace(None)
    with pytest.raises(binding.BnnError) as e:
        ctx.mlp_forward(net["desc"], dev(case["X"]), 4)
    assert e.value.status == -3


def test_two_streams_same_result(ctx):
    A, B = wl.gemm_case(300, 300, 1000, seed=12)
    want = oracle.gemm(A, B)
    s = torch.cuda.Stream()
    c2 = binding.Context(0, stream=s)
    with torch.cuda.stream(s):
        Ap = c2.pack_signs(dev(A, torch.int8))
        Bp = c2.pack_signs(dev(B, torch.int8), pack_along=1)
        r = [c2.xnor_gemm(Ap, Bp, 300, 300, 1000) for _ in range(2)]
    s.synchronize()
    for t in r:
        assert np.array_equal(t.cpu().numpy(), want)
    c2.close()
