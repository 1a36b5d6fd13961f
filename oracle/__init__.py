"""CPU oracle for the run-time path of a Binarized Neural Network (test infrastructure).

This package is NOT part of the product.  It holds the plain definition of what the
GPU library computes, on unpacked values (+1/-1 as int8, inputs as uint8), and is
called only by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark.  It imports nothing from the GPU package and the GPU package imports
nothing from here.

The arithmetic lives in ``bnn_oracle.c`` (plain C loops); this module compiles it
with gcc on first use and exposes numpy-in / numpy-out wrappers.  The only
arithmetic written in Python here is the composition of those calls into the layer
sequence of Algorithm 4 ("Running a BNN") and of the CIFAR-shaped ConvNet.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bnn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

# -ffp-contract=off: BatchNorm is defined as separate IEEE double operations.
_CFLAGS = ["-O3", "-march=native", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-std=c11"]


def build(force: bool = False) -> str:
    """Compile the oracle's C source into ``liboracle.so`` beside it (gcc)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.run(["gcc", *_CFLAGS, _SRC, "-o", tmp, "-lm"], check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        for name in (
            "oracle_sign_f32", "oracle_sign_i32", "oracle_gemm", "oracle_first_layer",
            "oracle_first_layer_bitplanes", "oracle_batchnorm", "oracle_sign_batchnorm",
            "oracle_threshold", "oracle_conv3x3", "oracle_conv3x3_u8", "oracle_maxpool2x2",
        ):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def host_threads() -> int:
    """Number of host threads the OpenMP loops will use (the affinity mask of this process)."""
    n = len(os.sched_getaffinity(0))
    env = os.environ.get("OMP_NUM_THREADS")
    return min(n, int(env)) if env else n


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _i64(v) -> ctypes.c_int64:
    return ctypes.c_int64(int(v))


def _check_pm1(a: np.ndarray, what: str) -> None:
    if a.size and not np.all((a == 1) | (a == -1)):
        raise ValueError(f"{what} must hold only -1 and +1")


# --------------------------------------------------------------------------- Eq. 1
def sign(x) -> np.ndarray:
    """Eq. 1: Sign(x) = +1 if x >= 0 else -1, as int8.  Accepts float32 or int32 arrays."""
    x = np.asarray(x)
    out = np.empty(x.shape, dtype=np.int8)
    if np.issubdtype(x.dtype, np.integer):
        xi = _c(x, np.int32)
        _load().oracle_sign_i32(_p(xi), _p(out), _i64(xi.size))
    else:
        xf = _c(x, np.float32)
        if np.isnan(xf).any():
            raise ValueError("Sign of NaN is not defined")
        _load().oracle_sign_f32(_p(xf), _p(out), _i64(xf.size))
    return out


# --------------------------------------------------------------------------- Section 4
def gemm(A, B) -> np.ndarray:
    """Section 4: ordinary integer product of two +-1 matrices, A (M x K) @ B (K x N) -> int32."""
    A = _c(A, np.int8)
    B = _c(B, np.int8)
    _check_pm1(A, "A")
    _check_pm1(B, "B")
    M, K = A.shape
    K2, N = B.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    C = np.zeros((M, N), dtype=np.int32)
    if M and N:
        _load().oracle_gemm(_p(A), _p(B), _p(C), _i64(M), _i64(N), _i64(K))
    return C


# --------------------------------------------------------------------------- Section 1.6
def first_layer(X, W) -> np.ndarray:
    """Eq. 6: s = x . w for 8-bit unsigned inputs X (M x K) and +-1 weights W (K x N) -> int32."""
    X = _c(X, np.uint8)
    W = _c(W, np.int8)
    _check_pm1(W, "W")
    M, K = X.shape
    K2, N = W.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    S = np.zeros((M, N), dtype=np.int32)
    if M and N:
        _load().oracle_first_layer(_p(X), _p(W), _p(S), _i64(M), _i64(N), _i64(K))
    return S


def first_layer_bitplanes(X, W) -> np.ndarray:
    """Eq. 7 / Algorithm 4 step 1: sum over the 8 bit-planes of 2^(n-1) (x^n . w), x^n in {0,1}."""
    X = _c(X, np.uint8)
    W = _c(W, np.int8)
    _check_pm1(W, "W")
    M, K = X.shape
    K2, N = W.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    S = np.zeros((M, N), dtype=np.int32)
    if M and N:
        _load().oracle_first_layer_bitplanes(_p(X), _p(W), _p(S), _i64(M), _i64(N), _i64(K))
    return S


# --------------------------------------------------------------------------- Algorithm 4: BatchNorm, Sign
def _bn_params(bn, N):
    gamma, beta, mean, var = (_c(bn[k], np.float32) for k in ("gamma", "beta", "mean", "var"))
    for v in (gamma, beta, mean, var):
        if v.shape != (N,):
            raise ValueError("BatchNorm parameter of wrong length")
    return gamma, beta, mean, var, float(bn.get("eps", 1e-4))


def batchnorm(S, bn) -> np.ndarray:
    """Run-time BatchNorm in float64 on integer pre-activations S (.. x N), per last-axis channel:
    y = gamma * ((s - mean) / sqrt(var + eps)) + beta (Algorithm 4, output layer)."""
    S = _c(S, np.int32)
    N = S.shape[-1]
    gamma, beta, mean, var, eps = _bn_params(bn, N)
    Y = np.zeros(S.shape, dtype=np.float64)
    if S.size:
        _load().oracle_batchnorm(_p(S), _p(gamma), _p(beta), _p(mean), _p(var), ctypes.c_double(eps), _p(Y),
                                 _i64(S.size // N), _i64(N))
    return Y


def sign_batchnorm(S, bn) -> np.ndarray:
    """Algorithm 4, hidden layers: Sign(BatchNorm(s, theta)) as int8 +-1."""
    S = _c(S, np.int32)
    N = S.shape[-1]
    gamma, beta, mean, var, eps = _bn_params(bn, N)
    out = np.zeros(S.shape, dtype=np.int8)
    if S.size:
        _load().oracle_sign_batchnorm(_p(S), _p(gamma), _p(beta), _p(mean), _p(var), ctypes.c_double(eps),
                                      _p(out), _i64(S.size // N), _i64(N))
    return out


def threshold(S, thr, flip=None) -> np.ndarray:
    """Integer decision rule of a hidden layer: +1 iff (s >= thr[n]) != flip[n], as int8 +-1."""
    S = _c(S, np.int32)
    N = S.shape[-1]
    thr = _c(thr, np.int32)
    if thr.shape != (N,):
        raise ValueError("thr of wrong length")
    f = None
    if flip is not None:
        f = _c(flip, np.uint8)
        if f.shape != (N,):
            raise ValueError("flip of wrong length")
    out = np.zeros(S.shape, dtype=np.int8)
    if S.size:
        _load().oracle_threshold(_p(S), _p(thr), _p(f) if f is not None else None, _p(out), _i64(S.size // N),
                                 _i64(N))
    return out


# --------------------------------------------------------------------------- Section 3.3: convolution
def conv3x3(act, wgt) -> np.ndarray:
    """3x3, stride 1, pad 1 convolution; taps outside the image contribute 0.
    act: B x H x W x Cin (int8 +-1, or uint8 for the first layer); wgt: Cout x 3 x 3 x Cin (+-1).
    Returns B x H x W x Cout int32."""
    act = np.ascontiguousarray(act)
    wgt = _c(wgt, np.int8)
    _check_pm1(wgt, "wgt")
    B, H, W, Cin = act.shape
    Cout = wgt.shape[0]
    if wgt.shape != (Cout, 3, 3, Cin):
        raise ValueError("wgt must be Cout x 3 x 3 x Cin")
    out = np.zeros((B, H, W, Cout), dtype=np.int32)
    if out.size == 0:
        return out
    args = (_p(wgt), _p(out), _i64(B), _i64(H), _i64(W), _i64(Cin), _i64(Cout))
    if act.dtype == np.uint8:
        _load().oracle_conv3x3_u8(_p(act), *args)
    else:
        act = _c(act, np.int8)
        _check_pm1(act, "act")
        _load().oracle_conv3x3(_p(act), *args)
    return out


def maxpool2x2(S) -> np.ndarray:
    """2x2 / stride 2 max-pooling of integer maps B x H x W x C (H, W even)."""
    S = _c(S, np.int32)
    B, H, W, C = S.shape
    if H % 2 or W % 2:
        raise ValueError("H and W must be even")
    out = np.zeros((B, H // 2, W // 2, C), dtype=np.int32)
    if out.size:
        _load().oracle_maxpool2x2(_p(S), _p(out), _i64(B), _i64(H), _i64(W), _i64(C))
    return out


# --------------------------------------------------------------------------- Algorithm 4, whole networks
def mlp_forward(X, weights, bns):
    """Algorithm 4 ("Running a BNN") for an MLP.

    X: batch x K0 uint8.  weights[k]: K_k x N_k int8 +-1 (k = 0..L-1).  bns[k]: BatchNorm
    parameters of layer k (dict with gamma, beta, mean, var, eps).
    Returns (scores float64 batch x N_L, [binary activations of every hidden layer as int8 +-1]).
    """
    L = len(weights)
    hidden = []
    s = first_layer(X, weights[0])                      # step 1 (Eq. 6)
    a = sign_batchnorm(s, bns[0])
    hidden.append(a)
    for k in range(1, L - 1):                           # step 2
        s = gemm(a, weights[k])
        a = sign_batchnorm(s, bns[k])
        hidden.append(a)
    s = gemm(a, weights[L - 1])                         # step 3: real-valued output
    return batchnorm(s, bns[L - 1]), hidden


def convnet_forward(X, layers):
    """CIFAR-shaped binarized ConvNet: each layer is conv3x3 -> optional 2x2 max-pool of the
    integer sums -> Sign(BatchNorm).  X: B x H x W x C uint8 (NHWC).
    layers: list of dicts {wgt, bn, pool}.  Returns the list of every layer's +-1 output (int8, NHWC)."""
    outs = []
    a = X
    for layer in layers:
        s = conv3x3(a, layer["wgt"])
        if layer.get("pool"):
            s = maxpool2x2(s)
        a = sign_batchnorm(s, layer["bn"])
        outs.append(a)
    return outs
