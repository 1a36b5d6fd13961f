"""Pins for the CPU oracle: each oracle function is checked against something other than itself --
hand-worked values, closed forms, invariants, independent library routines (numpy integer matmul,
torch conv2d / max_pool2d / batch_norm on CPU) and brute force in pure Python on tiny inputs."""
import itertools
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import workloads as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "handworked.json")))
RNG = np.random.default_rng(1234)


# ------------------------------------------------------------------ Eq. 1
def test_sign_handworked_and_zero_is_plus_one():
    g = GOLD["sign"]
    assert oracle.sign(np.array(g["x"], dtype=np.float32)).tolist() == g["s"]
    assert oracle.sign(np.array([0, -1, 1, -2**31, 2**31 - 1], dtype=np.int32)).tolist() == [1, -1, 1, -1, 1]
    with pytest.raises(ValueError):
        oracle.sign(np.array([np.nan], dtype=np.float32))


# ------------------------------------------------------------------ Section 4: binary GEMM
def test_gemm_handworked():
    g = GOLD["gemm_2x3_3x2"]
    assert oracle.gemm(np.array(g["A"]), np.array(g["B"])).tolist() == g["C"]


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (2, 3, 31), (3, 2, 32), (33, 1, 33), (1, 33, 63), (5, 7, 64),
                                   (4, 4, 65), (3, 5, 100)])
def test_gemm_bruteforce_python(M, N, K):
    A, B = wl.gemm_case(M, N, K, seed=K * 1000 + M)
    C = oracle.gemm(A, B)
    for m in range(M):
        for n in range(N):
            assert C[m, n] == sum(int(A[m, k]) * int(B[k, n]) for k in range(K))


def test_gemm_equals_numpy_integer_matmul_nonsquare():
    # distinct M, N, K so that a transposed operand or swapped index cannot pass
    A, B = wl.gemm_case(37, 53, 129, seed=7)
    assert np.array_equal(oracle.gemm(A, B), A.astype(np.int64) @ B.astype(np.int64))
    A, B = wl.config1()
    assert np.array_equal(oracle.gemm(A, B), A.astype(np.int32) @ B.astype(np.int32))


def test_gemm_closed_forms():
    K = 77
    ones = np.ones((3, K), np.int8)
    assert (oracle.gemm(ones, np.ones((K, 4), np.int8)) == K).all()
    a = wl.pm1(RNG, (1, K))
    assert oracle.gemm(a, a.T)[0, 0] == K                 # a.a = K
    assert oracle.gemm(a, (-a).T)[0, 0] == -K             # a.(-a) = -K
    for j in (1, 5, 40):                                  # flipping j entries lowers a.a by 2j
        b = a.copy()
        b[0, :j] *= -1
        assert oracle.gemm(a, b.T)[0, 0] == K - 2 * j


def test_gemm_is_K_minus_twice_hamming_distance():
    # Eq. 8 counts agreements; the ordinary product must equal K - 2*Hamming(a, b)
    M, N, K = 6, 5, 45
    A, B = wl.gemm_case(M, N, K, seed=11)
    C = oracle.gemm(A, B)
    for m in range(M):
        for n in range(N):
            hamming = sum(1 for k in range(K) if A[m, k] != B[k, n])
            agree = K - hamming
            assert C[m, n] == K - 2 * hamming == 2 * agree - K


@pytest.mark.parametrize("K", [1, 31, 32, 33, 100, 513])
def test_gemm_parity_and_bound(K):
    A, B = wl.gemm_case(16, 16, K, seed=K)
    C = oracle.gemm(A, B)
    assert ((C - K) % 2 == 0).all()
    assert (np.abs(C) <= K).all()


def test_gemm_statistics_iid():
    K = 256
    A, B = wl.gemm_case(256, 256, K, seed=3)
    C = oracle.gemm(A, B).astype(np.float64)
    assert abs(C.mean()) < 0.5                     # std of the mean = 16/256
    assert abs((C ** 2).mean() / K - 1.0) < 0.05


def test_gemm_empty_and_input_check():
    assert oracle.gemm(np.zeros((0, 5), np.int8), np.ones((5, 3), np.int8)).shape == (0, 3)
    assert (oracle.gemm(np.ones((2, 0), np.int8), np.ones((0, 3), np.int8)) == 0).all()
    with pytest.raises(ValueError):
        oracle.gemm(np.zeros((2, 2), np.int8), np.ones((2, 2), np.int8))


# ------------------------------------------------------------------ thresholds, BatchNorm, Sign
def test_threshold_extremes_ties_and_parity():
    K = 40
    A, B = wl.gemm_case(9, 12, K, seed=5)
    S = oracle.gemm(A, B)
    N = S.shape[1]
    assert (oracle.threshold(S, np.full(N, K + 1, np.int32)) == -1).all()
    assert (oracle.threshold(S, np.full(N, -K, np.int32)) == 1).all()
    assert (oracle.threshold(S, np.full(N, -K, np.int32), np.ones(N, np.uint8)) == -1).all()
    # tie s == thr -> +1 (Eq. 1 on s - thr)
    assert (oracle.threshold(S, S[0].copy())[0] == 1).all()
    # s = K (mod 2): thresholds t and t+1 give the same bits when t != K (mod 2)
    t = np.full(N, 3, np.int32)
    assert np.array_equal(oracle.threshold(S, t), oracle.threshold(S, t + 1))
    # and differ somewhere for t = K (mod 2) if some s == t
    t = S[3].copy()
    assert not np.array_equal(oracle.threshold(S, t), oracle.threshold(S, t + 1))
    # brute force
    thr = RNG.integers(-10, 10, N).astype(np.int32)
    flip = RNG.integers(0, 2, N).astype(np.uint8)
    out = oracle.threshold(S, thr, flip)
    for m, n in itertools.product(range(S.shape[0]), range(N)):
        assert out[m, n] == (1 if ((S[m, n] >= thr[n]) != bool(flip[n])) else -1)


def _bn(n, **kw):
    d = {"gamma": np.ones(n, np.float32), "beta": np.zeros(n, np.float32), "mean": np.zeros(n, np.float32),
         "var": np.ones(n, np.float32), "eps": 0.0}
    d.update(kw)
    return d


def test_batchnorm_special_cases():
    S = np.arange(-6, 7, dtype=np.int32).reshape(1, -1).repeat(3, 0).T.copy()   # 13 x 3
    n = 3
    assert np.array_equal(oracle.batchnorm(S, _bn(n)), S.astype(np.float64))    # identity parameters
    assert np.array_equal(oracle.sign_batchnorm(S, _bn(n)), np.where(S >= 0, 1, -1))
    # x == mean -> beta exactly
    Y = oracle.batchnorm(np.full((1, n), 5, np.int32), _bn(n, mean=np.full(n, 5, np.float32),
                                                           beta=np.array([0.25, -0.5, 0], np.float32)))
    assert Y.tolist() == [[0.25, -0.5, 0.0]]
    # var = 4 halves, gamma = -2 negates and doubles: y = -(x)
    Y = oracle.batchnorm(S, _bn(n, var=np.full(n, 4, np.float32), gamma=np.full(n, -2, np.float32)))
    assert np.array_equal(Y, -S.astype(np.float64))
    # gamma < 0 flips the sign rule; at x == mean the value is beta = 0 -> +1 (tie)
    out = oracle.sign_batchnorm(S, _bn(n, gamma=np.full(n, -1, np.float32)))
    assert np.array_equal(out, np.where(S <= 0, 1, -1))
    # gamma == 0 -> constant Sign(beta), with Sign(0) = +1
    out = oracle.sign_batchnorm(S, _bn(n, gamma=np.zeros(n, np.float32), beta=np.array([-1, 0, 1], np.float32)))
    assert (out == np.array([-1, 1, 1])).all()
    # eps is added under the square root: var = 0, eps = 4 -> divide by 2
    Y = oracle.batchnorm(S, _bn(n, var=np.zeros(n, np.float32), eps=4.0))
    assert np.array_equal(Y, S / 2.0)


def test_batchnorm_matches_torch_library_routine():
    n, M, K = 64, 50, 4096
    bn = wl.batchnorm_params(RNG, n, K)
    S = RNG.integers(-K, K + 1, (M, n)).astype(np.int32)
    Y = oracle.batchnorm(S, bn)
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    ref = torch.nn.functional.batch_norm(t(S), t(bn["mean"]), t(bn["var"]), t(bn["gamma"]), t(bn["beta"]),
                                         training=False, eps=bn["eps"]).numpy()
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12)
    sgn = oracle.sign_batchnorm(S, bn)
    clear = np.abs(ref) > 1e-9
    assert np.array_equal(sgn[clear], np.where(ref >= 0, 1, -1)[clear])
    assert np.array_equal(sgn, np.where(Y >= 0, 1, -1))


# ------------------------------------------------------------------ Section 1.6: first layer
def test_first_layer_handworked():
    g = GOLD["first_layer_bitplanes"]
    X = np.array([g["x"]], np.uint8)
    W = np.array(g["w"], np.int8).reshape(-1, 1)
    assert oracle.first_layer(X, W)[0, 0] == g["s"]
    assert oracle.first_layer_bitplanes(X, W)[0, 0] == g["s"]
    for p, d in enumerate(g["plane_dots_lsb_first"]):      # a single plane: x in {0, 2^p}
        Xp = ((X >> p) & 1).astype(np.uint8) << p
        assert oracle.first_layer(Xp, W)[0, 0] == d * (1 << p)


def test_first_layer_library_identity_and_special_cases():
    M, N, K = 13, 21, 100
    X = wl.u8(RNG, (M, K))
    W = wl.pm1(RNG, (K, N))
    S = oracle.first_layer(X, W)
    assert np.array_equal(S, X.astype(np.int64) @ W.astype(np.int64))
    assert np.array_equal(S, oracle.first_layer_bitplanes(X, W))          # Eq. 6 == Eq. 7
    assert (np.abs(S) <= 255 * K).all()
    assert np.array_equal(oracle.first_layer(np.full((2, K), 255, np.uint8), W),
                          np.tile(255 * W.astype(np.int64).sum(0), (2, 1)))
    assert (oracle.first_layer(np.zeros((2, K), np.uint8), W) == 0).all()


def test_first_layer_plane_reading():
    """Algorithm 4 writes the planes through XnorDotProduct, which would read a 0 bit as -1; that literal
    reading gives 2s - 255*sum(w), not s.  Eq. 6-7 (bits as 0/1) is the reading that yields x.w."""
    M, N, K = 4, 6, 50
    X = wl.u8(RNG, (M, K))
    W = wl.pm1(RNG, (K, N))
    s = oracle.first_layer(X, W).astype(np.int64)
    literal = np.zeros_like(s)
    for p in range(8):
        plane_pm1 = (2 * ((X >> p) & 1).astype(np.int8) - 1).astype(np.int8)
        literal += (1 << p) * oracle.gemm(plane_pm1, W)
    assert np.array_equal(literal, 2 * s - 255 * W.astype(np.int64).sum(0))


# ------------------------------------------------------------------ Section 3.3: convolution, pooling
def _torch_conv(act, wgt):
    a = torch.from_numpy(act.astype(np.float64)).permute(0, 3, 1, 2)
    w = torch.from_numpy(wgt.astype(np.float64)).permute(0, 3, 1, 2)
    return torch.nn.functional.conv2d(a, w, padding=1).permute(0, 2, 3, 1).numpy()


@pytest.mark.parametrize("B,H,W,Cin,Cout", [(2, 5, 7, 32, 9), (1, 1, 1, 64, 3), (1, 2, 2, 3, 4), (2, 4, 4, 5, 6)])
def test_conv_matches_torch_zero_padding(B, H, W, Cin, Cout):
    act = wl.pm1(RNG, (B, H, W, Cin))
    wgt = wl.pm1(RNG, (Cout, 3, 3, Cin))
    out = oracle.conv3x3(act, wgt)
    assert np.array_equal(out, _torch_conv(act, wgt).astype(np.int64))
    actu = wl.u8(RNG, (B, H, W, Cin))
    assert np.array_equal(oracle.conv3x3(actu, wgt), _torch_conv(actu, wgt).astype(np.int64))


def test_conv_closed_forms_and_parity():
    g = GOLD["conv_corner"]
    out = oracle.conv3x3(np.ones((1, g["H"], g["W"], 1), np.int8), np.ones((1, 3, 3, 1), np.int8))
    assert (out == g["value"]).all()
    B, H, W, Cin, Cout = 1, 6, 5, 32, 7
    wgt = wl.pm1(RNG, (Cout, 3, 3, Cin))
    act = wl.pm1(RNG, (B, H, W, Cin))
    out = oracle.conv3x3(act, wgt)
    ys, xs = np.arange(H), np.arange(W)
    ny = 3 - (ys == 0) - (ys == H - 1)
    nx = 3 - (xs == 0) - (xs == W - 1)
    kvalid = Cin * ny[:, None] * nx[None, :]
    assert ((out[0] - kvalid[:, :, None]) % 2 == 0).all()         # dot = K_valid (mod 2)
    assert (np.abs(out[0]) <= kvalid[:, :, None]).all()
    # all-ones image: every output is the sum of the weights under the valid taps
    ones = oracle.conv3x3(np.ones((1, H, W, Cin), np.int8), wgt)
    w64 = wgt.astype(np.int64)
    assert np.array_equal(ones[0, 0, 0], w64[:, 1:, 1:, :].sum((1, 2, 3)))          # top-left corner
    assert np.array_equal(ones[0, 2, 2], w64.sum((1, 2, 3)))                        # interior
    assert np.array_equal(ones[0, H - 1, 2], w64[:, :2, :, :].sum((1, 2, 3)))       # bottom edge
    # interior pixels are a GEMM of the im2col matrix
    patches = np.stack([act[0, y - 1:y + 2, x - 1:x + 2, :].reshape(-1) for y in range(1, H - 1)
                        for x in range(1, W - 1)])
    ref = oracle.gemm(patches, wgt.reshape(Cout, -1).T.copy())
    assert np.array_equal(out[0, 1:H - 1, 1:W - 1, :].reshape(-1, Cout), ref)


def test_maxpool_matches_torch_and_or_of_bits_identity():
    S = RNG.integers(-50, 50, (2, 6, 4, 5)).astype(np.int32)
    P = oracle.maxpool2x2(S)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(S.astype(np.float64)).permute(0, 3, 1, 2), 2)
    assert np.array_equal(P, ref.permute(0, 2, 3, 1).numpy().astype(np.int64))
    # threshold of the max == OR over the window of thresholded values (thr form), also with flip
    thr = RNG.integers(-20, 20, 5).astype(np.int32)
    for flip in (None, RNG.integers(0, 2, 5).astype(np.uint8)):
        pooled_then_thr = oracle.threshold(P, thr, flip)
        q = oracle.threshold(S, thr) > 0                                   # plain (s >= thr)
        ored = q[:, 0::2, 0::2] | q[:, 0::2, 1::2] | q[:, 1::2, 0::2] | q[:, 1::2, 1::2]
        f = np.zeros(5, bool) if flip is None else flip.astype(bool)
        assert np.array_equal(pooled_then_thr > 0, ored ^ f)


# ------------------------------------------------------------------ Algorithm 4 end to end
def test_mlp_forward_is_algorithm4_composed_from_library_routines():
    case = wl.mlp_case(batch=9, sizes=(50, 64, 40, 10), seed=21)
    scores, hidden = oracle.mlp_forward(case["X"], case["weights"], case["bns"])
    t = lambda a: torch.from_numpy(np.asarray(a)).double()

    def bn(s, p):
        return torch.nn.functional.batch_norm(t(s), t(p["mean"]), t(p["var"]), t(p["gamma"]), t(p["beta"]),
                                              training=False, eps=p["eps"]).numpy()
    a = case["X"].astype(np.int64)
    for k, (Wk, p) in enumerate(zip(case["weights"], case["bns"])):
        s = a @ Wk.astype(np.int64)
        y = bn(s, p)
        if k < len(case["weights"]) - 1:
            assert np.abs(y).min() > 1e-9, "test case sits on a tie; change the seed"
            a = np.where(y >= 0, 1, -1)
            assert np.array_equal(hidden[k], a)
        else:
            assert np.allclose(scores, y, rtol=1e-12, atol=1e-12)
    assert len(hidden) == 2 and scores.shape == (9, 10)


def test_convnet_forward_composition():
    case = wl.convnet_case(batch=2, hw=8, channels=(32, 32, 64, 64), seed=5)
    outs = oracle.convnet_forward(case["X"], case["layers"])
    assert [o.shape for o in outs] == [(2, 8, 8, 32), (2, 4, 4, 32), (2, 4, 4, 64), (2, 2, 2, 64)]
    a = case["X"]
    for layer, o in zip(case["layers"], outs):
        s = _torch_conv(a, layer["wgt"]).astype(np.int64)
        if layer["pool"]:
            s = torch.nn.functional.max_pool2d(torch.from_numpy(s.astype(np.float64)).permute(0, 3, 1, 2),
                                               2).permute(0, 2, 3, 1).numpy().astype(np.int64)
        y = oracle.batchnorm(s.astype(np.int32), layer["bn"])
        a = np.where(y >= 0, 1, -1).astype(np.int8)
        assert np.array_equal(o, a)


def test_workloads_are_seeded_and_shaped():
    A, B = wl.config1()
    A2, B2 = wl.config1()
    assert A.shape == (64, 512) and B.shape == (512, 256) and np.array_equal(A, A2) and np.array_equal(B, B2)
    assert set(np.unique(A)) == {-1, 1}
    d1, d2 = wl.dense_case(1, 64, 32), wl.dense_case(16, 64, 32)
    assert np.array_equal(d1["W"], d2["W"]) and np.array_equal(d1["thr"], d2["thr"])
    assert d1["thr"].min() >= -64 and d1["thr"].max() <= 64
