"""Seeded synthetic inputs shaped like the paper's workloads.

This module only DRAWS numbers (numpy PCG64, fixed draw order) and fixes shapes.  It holds
none of the method's arithmetic: no packing, no popcount, no BatchNorm evaluation, no
thresholds derived from BatchNorm.  Both the CPU oracle's tests and the GPU tests feed
on the same arrays produced here; MNIST / CIFAR-10 themselves are not available, so
uniform random pixels of the same shape and range stand in for them.

Draw order inside every workload: weights (layer order) -> BatchNorm parameters per layer
(gamma, beta, mean, var) -> integer thresholds (if any) -> inputs.
"""
from __future__ import annotations

import numpy as np


def pm1(rng: np.random.Generator, shape) -> np.ndarray:
    """iid +-1 with P(+1) = 0.5, as int8."""
    return (2 * rng.integers(0, 2, size=shape, dtype=np.int8) - 1).astype(np.int8)


def u8(rng: np.random.Generator, shape) -> np.ndarray:
    """iid uniform 0..255, as uint8 (stand-in for image pixels)."""
    return rng.integers(0, 256, size=shape, dtype=np.uint8)


def batchnorm_params(rng: np.random.Generator, n: int, K: int, eps: float = 1e-4) -> dict:
    """gamma ~ N(1, 0.1), beta ~ N(0, 0.1), running mean ~ N(0, sqrt(K)/4), running var ~ U(0.5, 2) * K
    (second argument of N(.,.) is the standard deviation); float32."""
    return {
        "gamma": rng.normal(1.0, 0.1, n).astype(np.float32),
        "beta": rng.normal(0.0, 0.1, n).astype(np.float32),
        "mean": rng.normal(0.0, np.sqrt(K) / 4.0, n).astype(np.float32),
        "var": (rng.uniform(0.5, 2.0, n) * K).astype(np.float32),
        "eps": eps,
    }


def gemm_case(M: int, N: int, K: int, seed: int):
    """One binary matrix product: A (M x K) and B (K x N), iid +-1."""
    rng = np.random.default_rng(seed)
    return pm1(rng, (M, K)), pm1(rng, (K, N))


def config1():
    """Single small binary GEMM: 64 x 512 times 512 x 256, seed 0."""
    return gemm_case(64, 256, 512, seed=0)


GEMM_SWEEP = [(4096, 4096, 4096), (8192, 8192, 8192), (16384, 16384, 16384), (8192, 8192, 4100)]


def mlp_case(batch: int = 10000, sizes=(784, 4096, 4096, 4096, 10), seed: int = 1):
    """MNIST-shaped MLP (Section 2.1: three hidden layers of 4096 binary units, 10 outputs).

    sizes = (inputs, hidden..., outputs).  Returns dict with
      weights: list of K_k x N_k int8 +-1,  bns: list of BatchNorm parameter dicts,  X: batch x inputs uint8."""
    rng = np.random.default_rng(seed)
    weights = [pm1(rng, (sizes[i], sizes[i + 1])) for i in range(len(sizes) - 1)]
    bns = [batchnorm_params(rng, sizes[i + 1], sizes[i]) for i in range(len(sizes) - 1)]
    X = u8(rng, (batch, sizes[0]))
    return {"weights": weights, "bns": bns, "X": X, "sizes": tuple(sizes), "batch": batch}


CONVNET_CHANNELS = (128, 128, 256, 256, 512, 512)


def convnet_case(batch: int = 256, hw: int = 32, in_ch: int = 3, channels=CONVNET_CHANNELS, seed: int = 3):
    """CIFAR-shaped binarized ConvNet: 3x3 pad-1 convolutions of widths `channels`, a 2x2 max-pool
    after every second one; the first convolution takes the 8-bit image.
    Returns dict with layers: list of {wgt: Cout x 3 x 3 x Cin int8, bn: dict, pool: bool} and X: B x H x W x C uint8."""
    rng = np.random.default_rng(seed)
    cins = (in_ch,) + tuple(channels[:-1])
    wgts = [pm1(rng, (cout, 3, 3, cin)) for cin, cout in zip(cins, channels)]
    bns = [batchnorm_params(rng, cout, 9 * cin) for cin, cout in zip(cins, channels)]
    X = u8(rng, (batch, hw, hw, in_ch))
    layers = [{"wgt": w, "bn": b, "pool": (i % 2 == 1)} for i, (w, b) in enumerate(zip(wgts, bns))]
    return {"layers": layers, "X": X, "batch": batch, "hw": hw}


DENSE_BATCHES = (1, 16, 256, 4096, 65536)


def dense_case(batch: int, K: int = 4096, N: int = 4096, seed: int = 4):
    """One fused binary dense layer: activations batch x K, weights K x N, integer thresholds
    uniform in [-64, 64].  The weights and thresholds do not depend on `batch`."""
    rng = np.random.default_rng(seed)
    W = pm1(rng, (K, N))
    thr = rng.integers(-64, 65, size=N, dtype=np.int32)
    A = pm1(np.random.default_rng([seed, batch]), (batch, K))
    return {"A": A, "W": W, "thr": thr}


def dictionary_conv_weights(rng: np.random.Generator, Cout: int, Cin: int, distinct_per_channel: int) -> np.ndarray:
    """Cout x 3 x 3 x Cin +-1 weights with repeated 2-D filters (Section 3.3 reports that only 42 % of a trained network's
    filters are distinct): in every input channel the Cout 3x3 slices are drawn from `distinct_per_channel` random patterns
    (distinct even up to negation, each used at least once), with random signs.  Stands in for trained weights."""
    wgt = np.empty((Cout, 3, 3, Cin), np.int8)
    for c in range(Cin):
        codes = rng.choice(256, size=distinct_per_channel, replace=False)      # classes up to sign: tap 0 = +1, 8 free taps
        pats = np.array([[1] + [1 if (k >> b) & 1 else -1 for b in range(8)] for k in codes], np.int8)
        pick = np.concatenate([np.arange(distinct_per_channel), rng.integers(0, distinct_per_channel, Cout - distinct_per_channel)])
        rng.shuffle(pick)
        sign = (2 * rng.integers(0, 2, Cout) - 1).astype(np.int8)
        wgt[:, :, :, c] = (pats[pick] * sign[:, None]).reshape(Cout, 3, 3)
    return wgt
