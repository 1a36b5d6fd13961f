"""Uploading a network to the GPU through the C ABI: weights are sign-packed by bnn_pack_signs,
BatchNorm + Sign is folded into integer thresholds by bnn_fold_batchnorm, and the layer list is laid
out as the descriptor bnn_mlp_forward takes.  Everything numeric happens inside the library calls."""
from __future__ import annotations

import numpy as np
import torch

from . import binding


def _dev(ctx, a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(f"cuda:{ctx.device}")


def pack_weight(ctx, W: np.ndarray) -> torch.Tensor:
    """K x N int8 +-1 host matrix -> packed N x K device operand."""
    return ctx.pack_signs(_dev(ctx, W, torch.int8), pack_along=1)


def fold(ctx, bn: dict, x_max: int):
    thr, flip = binding.fold_batchnorm(*(torch.from_numpy(np.asarray(bn[k])) for k in ("gamma", "beta", "mean", "var")),
                                       bn["eps"], x_max)
    return thr.to(f"cuda:{ctx.device}"), flip.to(f"cuda:{ctx.device}")


def prepare_mlp(ctx, weights, bns, expand_weights: bool = True):
    """Algorithm 4's inputs (binary weights W^b and BatchNorm parameters theta) -> device layer list.
    With expand_weights the hidden layers' weights are also stored as +-1 bytes (bnn_expand_signs) once, so the
    tensor-core engine does not have to expand them on every forward call."""
    layers = []
    L = len(weights)
    for k, (W, bn) in enumerate(zip(weights, bns)):
        K, N = W.shape
        d = {"Wp": pack_weight(ctx, W), "K": K, "N": N}
        if k < L - 1:
            d["thr"], d["flip"] = fold(ctx, bn, 255 * K if k == 0 else K)
            if expand_weights:
                # the first layer multiplies bytes by bytes; the others can run on either operand width
                d["W8"] = ctx.expand_signs(d["Wp"], N, K)
                if k > 0:
                    d["W4"] = ctx.expand_signs_f4(d["Wp"], N, K)
        else:
            for name in ("gamma", "beta", "mean", "var"):
                d[name] = _dev(ctx, bn[name], torch.float32)
            d["eps"] = bn["eps"]
        layers.append(d)
    desc, keep = ctx.make_mlp_desc(layers)
    return {"layers": layers, "desc": desc, "_keep": keep}


def prepare_convnet(ctx, layers, expand_weights: bool = True):
    """Conv layer list {wgt: Cout x 3 x 3 x Cin, bn, pool} -> packed device weights and folded thresholds
    (and, with expand_weights, the weights as +-1 bytes and, where used, 4-bit nibbles for the tensor-core engine)."""
    out = []
    for i, L in enumerate(layers):
        wgt = L["wgt"]
        Cout, _, _, Cin = wgt.shape
        flat = wgt.reshape(Cout, 9 * Cin)                      # [n][tap*Cin + c]
        if i == 0 and 9 * Cin <= 32:
            Wp = ctx.pack_signs(_dev(ctx, flat, torch.int8), pack_along=0)[:, 0].contiguous()
            x_max = 255 * 9 * Cin
        else:
            Wp = ctx.pack_signs(_dev(ctx, flat, torch.int8), pack_along=0)[:, :9 * Cin // 32].contiguous()
            x_max = 9 * Cin
        thr, flip = fold(ctx, L["bn"], x_max)
        d = {"Wp": Wp, "Cin": Cin, "Cout": Cout, "pool": bool(L.get("pool")), "thr": thr, "flip": flip}
        if expand_weights:
            # the same bits viewed as Cout rows of 9*Cin: re-pack with a legal leading dimension, then expand
            rows = ctx.pack_signs(_dev(ctx, flat, torch.int8), pack_along=0)
            d["W8"] = ctx.expand_signs(rows, Cout, 9 * Cin)
            if i > 0 and Cin % 128 == 0:                       # layers the library may run on 4-bit operands
                d["W4"] = ctx.expand_signs_f4(rows, Cout, 9 * Cin)
        out.append(d)
    return out


def convnet_output_shape(net, B: int, H: int, W: int):
    for L in net:
        if L["pool"]:
            H, W = H // 2, W // 2
    return (B, H, W, binding.words(net[-1]["Cout"]))


def convnet_forward(ctx, net, X_u8: torch.Tensor, keep_all: bool = False):
    """X_u8: B x H x W x C uint8 on the device.  One bnn_binary_conv2d call per layer; returns the packed
    output of the last layer (or of every layer)."""
    B, H, W, _ = X_u8.shape
    act = X_u8
    outs = []
    for L in net:
        act, _ = ctx.binary_conv2d(act, B, H, W, L["Cin"], L["Wp"], L["Cout"], pool=L["pool"], thr=L["thr"],
                                   flip=L["flip"])
        if L["pool"]:
            H, W = H // 2, W // 2
        if keep_all:
            outs.append(act)
    return outs if keep_all else act


def convnet_workspace_bytes(ctx, net, B: int, H: int, W: int) -> int:
    """Largest workspace any layer of `net` asks for on the tensor-core engine (0 if none qualifies)."""
    need = 0
    for L in net:
        need = max(need, ctx.conv_workspace_bytes(B, H, W, L["Cin"], L["Cout"], L["pool"]))
        if L["pool"]:
            H, W = H // 2, W // 2
    return need
