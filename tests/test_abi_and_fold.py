"""CPU-side checks of the product's boundary: the shared library builds, loads and exports every function
the header declares; status strings; and the host helper that folds BatchNorm + Sign into an integer
threshold, compared with the oracle's double-precision Sign(BatchNorm(x)) over every integer x."""
import os
import re

import numpy as np
import pytest
import torch

import oracle
from paper_1602_02830_b200 import binding, build, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bnn_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bnn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function(lib):
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert lib.bnn_status_string(0) == b"ok"
    seen = {lib.bnn_status_string(s) for s in range(-6, 1)}
    assert len(seen) == 7


def test_host_argument_errors_need_no_gpu(lib):
    # NULL context / NULL output are rejected before any CUDA call
    assert lib.bnn_destroy(None) == -1
    assert lib.bnn_set_popc_variant(None, 0) == -1
    assert lib.bnn_xnor_gemm(None, None, 0, None, 0, None, 0, 1, 1, 1) == -1
    assert lib.bnn_fold_batchnorm(None, None, None, None, 0.0, 4, 10, None, None) == -1
    assert lib.bnn_fold_batchnorm(None, None, None, None, 0.0, 0, 10, None, None) == 0


def _fake_mlp_desc(ldw_first=28, ptr=0x1000, wp_first=None):
    """A two-layer descriptor whose pointers are never dereferenced (every call below fails, or only sizes things)."""
    arr = (binding.LayerDesc * 2)()
    arr[0].Wp, arr[0].ldw_w, arr[0].K, arr[0].N, arr[0].thr = (wp_first or ptr), ldw_first, 784, 256, ptr
    arr[1].Wp, arr[1].ldw_w, arr[1].K, arr[1].N = ptr, 8, 256, 10
    arr[1].gamma = arr[1].beta = arr[1].mean = arr[1].var = ptr
    return binding.MlpDesc(2, arr), arr


def test_mlp_descriptor_layout_errors_need_no_gpu(lib):
    """A packed weight matrix with an odd or too small leading dimension, or a misaligned base, is refused by every MLP
    entry point before anything could be launched (the kernels read the rows with 128-bit loads)."""
    import ctypes
    good, keep = _fake_mlp_desc()
    assert lib.bnn_mlp_workspace_bytes(ctypes.byref(good), 100, 0) > 0
    calls = (lambda d: lib.bnn_mlp_forward(None, ctypes.byref(d), None, 784, 100, None, 10, None),
             lambda d: lib.bnn_mlp_forward_host(None, ctypes.byref(d), None, 784, 100, None, 10),
             lambda d: lib.bnn_mlp_forward_noalloc(None, ctypes.byref(d), None, 784, 100, None, 10))
    for bad_kwargs, status in (({"ldw_first": 25}, -2), ({"ldw_first": 27}, -2), ({"ldw_first": 24}, -1),
                               ({"wp_first": 0x1004}, -2)):
        bad, keep2 = _fake_mlp_desc(**bad_kwargs)
        assert lib.bnn_mlp_workspace_bytes(ctypes.byref(bad), 100, 0) == 0
        for call in calls:
            assert call(bad) == status
    for call in calls:
        assert call(good) == -1              # a sound descriptor gets as far as the missing context


def test_expand_layout_errors_need_no_gpu(lib):
    """bnn_expand_signs / _f4 read the packed source with 64- and 128-bit loads: the packed-matrix rule is enforced."""
    for fn in (lib.bnn_expand_signs, lib.bnn_expand_signs_f4):
        assert fn(None, 0x1000, 5, 8, 130, 0x2000) == -2      # odd leading dimension
        assert fn(None, 0x1000, 6, 8, 130, 0x2000) == -2      # not a multiple of 4 words
        assert fn(None, 0x1004, 8, 8, 130, 0x2000) == -2      # source only 4-byte aligned
        assert fn(None, 0x1000, 4, 8, 130, 0x2000) == -1      # leading dimension below ceil(K / 32)
        assert fn(None, 0x1000, 8, 8, 130, 0x2008) == -2      # destination not 16-byte aligned
        assert fn(None, 0x1000, 8, 8, 130, 0x2000) == -1      # sound layout: stops at the missing context
        assert fn(None, None, 0, 0, 130, None) == -1          # empty problem, still no context


def _fold_matches_oracle(bn, x_max):
    thr, flip = binding.fold_batchnorm(*(torch.from_numpy(bn[k]) for k in ("gamma", "beta", "mean", "var")),
                                       bn["eps"], x_max)
    n = bn["gamma"].size
    xs = np.arange(-x_max, x_max + 1, dtype=np.int32)
    S = np.repeat(xs[:, None], n, axis=1)
    want = oracle.sign_batchnorm(S, bn)                                   # double-precision definition
    f = np.array([(int(flip[c // 32]) >> (c % 32)) & 1 for c in range(n)], dtype=np.uint8)
    got = oracle.threshold(S, thr.numpy(), f)                             # integer rule with the folded values
    assert np.array_equal(got, want)
    assert thr.min() >= -x_max and thr.max() <= x_max + 1
    return thr.numpy(), f


def test_fold_batchnorm_random_channels():
    rng = np.random.default_rng(5)
    for K in (27, 784, 4096):
        _fold_matches_oracle(wl.batchnorm_params(rng, 96, K), K)


def test_fold_batchnorm_adversarial_channels():
    g = np.array([1, -1, 0, 0, 0, 2, -2, 1, -1, 1e-30, -1e-30, 1, -1, 3, 0.5, -0.5], np.float32)
    b = np.array([0, 0, -1, 0, 1, 4, 4, 1e6, 1e6, 0, 0, -1e6, -1e6, -7.5, 0.25, 0.25], np.float32)
    m = np.array([0, 0, 0, 0, 0, 3, 3, 0, 0, 5, 5, 0, 0, 2.5, -3, -3], np.float32)
    v = np.array([1, 1, 1, 1, 1, 4, 4, 1, 1, 1, 1, 1, 1, 9, 0.25, 0.25], np.float32)
    bn = {"gamma": g, "beta": b, "mean": m, "var": v, "eps": 0.0}
    thr, f = _fold_matches_oracle(bn, 40)
    assert thr[0] == 0 and f[0] == 0            # Sign(x): tie at 0 -> +1
    assert thr[1] == 1 and f[1] == 1            # Sign(-x): +1 iff x <= 0
    assert (thr[2], f[2]) == (-40, 1)           # gamma = 0, beta < 0 -> always -1
    assert (thr[3], f[3]) == (-40, 0)           # gamma = 0, beta = 0 -> always +1
    assert (thr[7], f[7]) == (-40, 0) and (thr[11], f[11]) == (41, 0)     # saturated
    assert (thr[8], f[8]) == (41, 1) and (thr[12], f[12]) == (-40, 1)
    _fold_matches_oracle({**bn, "eps": 1e-4}, 40)


def test_fold_rejects_bad_variance():
    one = torch.ones(1)
    with pytest.raises(binding.BnnError):
        binding.fold_batchnorm(one, one, one, -one, 0.0, 10)


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()


def test_test_side_packer_roundtrip():
    from util import np_pack_pm1, np_unpack_pm1, padding_is_zero
    x = wl.pm1(np.random.default_rng(0), (5, 70))
    p = np_pack_pm1(x, 4)
    assert p.shape == (5, 4) and np.array_equal(np_unpack_pm1(p, 70), x) and padding_is_zero(p, 70)
    assert np_pack_pm1(np.array([[1, -1, 1]]))[0, 0] == 0b101


@pytest.mark.parametrize("slots", [2, 3, 4, 5, 6, 7])
def test_operand_ring_gives_every_barrier_one_consumer(slots):
    """Ring arithmetic of the tensor-engine kernels, on the host.  Two threads take alternate stages; a wait on a phase
    parity is only right while the waiter is at most one phase ahead of its barrier, which holds when every barrier is
    waited on by ONE thread in phase order (that thread's own previous use is the phase before).  With one barrier per
    slot and an odd number of slots the uses of a barrier alternate between the threads; with two barrier pairs per slot
    they never do."""
    build.build()
    consumer_of, producer_of, last_phase = {}, {}, {}
    for G in range(0, 20 * slots + 3):
        r = binding.debug_ring_position(G, slots, 2)
        assert r["slot"] == G % slots
        assert r["barrier"] == G % (2 * slots) and r["parity"] == (G // (2 * slots)) % 2
        # one consuming thread (stage parity) per barrier, phases in order
        assert consumer_of.setdefault(r["barrier"], G % 2) == G % 2
        phase = G // (2 * slots)
        assert last_phase.get(r["barrier"], -1) == phase - 1
        last_phase[r["barrier"]] = phase
        # the producer refills a slot after the stage `slots` earlier was consumed: that stage's barrier and parity
        assert r["reuses"] == (1 if G >= slots else 0)
        if G >= slots:
            e = binding.debug_ring_position(G - slots, slots, 1)
            assert (r["prev_barrier"], r["prev_parity"]) == (e["barrier"], e["parity"])
            # with two producer threads on alternate stages, each "empty" barrier also has one waiting thread
            assert producer_of.setdefault(r["prev_barrier"], G % 2) == G % 2
        # advancing by the thread's stride lands where a fresh start would
        n = binding.debug_ring_position(G + 2, slots, 1)
        assert (r["next_barrier"], r["next_parity"]) == (n["barrier"], n["parity"])
    # the flawed layout for comparison: one barrier per slot, odd ring -> consecutive uses of a barrier change hands
    if slots % 2 == 1:
        users = [G % 2 for G in range(0, 4 * slots) if G % slots == 0]
        assert users[0] != users[1]


def test_operand_ring_position_rejects_bad_arguments():
    build.build()
    for args in ((0, 0, 1), (0, 3, 0), (0, 3, 7)):
        with pytest.raises(binding.BnnError):
            binding.debug_ring_position(*args)
