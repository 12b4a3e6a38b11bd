"""Synthetic workloads: shapes and value distributions of the benchmark configurations.

Everything is generated on the host as plain numpy arrays:
activations NHWC fp32, weights [Cout][KH][KW][Cin] fp32, masks uint8 of the
weight's shape.  These stand in for a trained, pruned MobileNet-v1 and for
feature maps of real images; only shapes, sparsity structure and value ranges
are reproduced.
"""
from __future__ import annotations

import math

import numpy as np

from . import masks as _masks
from .rng import STREAM_BIAS, STREAM_MASK, STREAM_W, STREAM_X, normal, uniform01


def single_conv_inputs(n, h, w, cin, cout, k, g, sparsity_pct, seed=0, w_sigma=0.05, b_sigma=0.05,
                       mask_mode="balanced", gi=1, layer=0):
    """One group-sparse k x k convolution layer (k = 1 or 3): activations U[0,1), weights and bias normal."""
    if cout % g:
        raise ValueError("cout must be a multiple of g")
    base = 16 * layer
    x = uniform01(seed, base + STREAM_X, n * h * w * cin).reshape(n, h, w, cin)
    wt = normal(seed, base + STREAM_W, cout * k * k * cin, w_sigma).reshape(cout, k, k, cin)
    b = normal(seed, base + STREAM_BIAS, cout, b_sigma)
    ngroups = cout // g
    if mask_mode == "balanced":
        um = _masks.group_mask_balanced(seed, base + STREAM_MASK, ngroups, cin, sparsity_pct, gi)
    elif mask_mode == "layer_global":
        um = _masks.group_mask_layer_global(seed, base + STREAM_MASK, ngroups, cin, sparsity_pct)
    elif mask_mode == "magnitude":
        um = _masks.group_mask_magnitude(wt, g, sparsity_pct)
    else:
        raise ValueError(mask_mode)
    return {"x": x, "w": wt, "bias": b, "mask": _masks.expand_mask(um, g, k, k), "unit_mask": um,
            "g": g, "sparsity_pct": sparsity_pct}


def config1(seed=0):
    """Single 1x1 layer, batch 1, 56x56, 64 -> 128, G=4, 50 % sparse."""
    return single_conv_inputs(1, 56, 56, 64, 128, 1, 4, 50, seed, 0.05, 0.05)


def config4(seed=0, n=32):
    """Group-sparse 3x3 layer, 28x28, 256 -> 256, G=4, half of the (group, channel) kernels removed."""
    return single_conv_inputs(n, 28, 28, 256, 256, 3, 4, 50, seed, 0.02, 0.02)


def config5(g, sparsity_pct, seed=0, n=256):
    """1x1 layer of the sparsity sweep: 14x14, 1024 -> 1024."""
    return single_conv_inputs(n, 14, 14, 1024, 1024, 1, g, sparsity_pct, seed, 0.02, 0.05)


def config5_family(cases, seed=0, n=256):
    """The layers of the sparsity sweep for several (g, sparsity_pct) pairs.  Activations, weights and bias do not
    depend on g or the sparsity (same streams, same seed), so they are drawn once and shared; only the masks differ.
    Yields the same dicts as config5(g, sparsity_pct, seed, n)."""
    base = None
    for g, sp in cases:
        if base is None:
            base = config5(g, sp, seed, n)
            yield base
            continue
        um = _masks.group_mask_balanced(seed, STREAM_MASK, 1024 // g, 1024, sp, 1)
        yield {"x": base["x"], "w": base["w"], "bias": base["bias"], "mask": _masks.expand_mask(um, g, 1, 1),
               "unit_mask": um, "g": g, "sparsity_pct": sp}


def mobilenet_v1_shapes():
    """Layer list of MobileNet-v1, width 1.0, 224x224x3 input (Howard et al. 2017, Table 1).

    Each entry: name, kind (conv0 | dw | pw | pool | fc), input side length,
    input channels, output channels, stride.
    """
    layers = [dict(name="conv0", kind="conv0", hin=224, cin=3, cout=32, stride=2)]
    chans = [(32, 64, 1), (64, 128, 2), (128, 128, 1), (128, 256, 2), (256, 256, 1), (256, 512, 2)] \
        + [(512, 512, 1)] * 5 + [(512, 1024, 2), (1024, 1024, 1)]
    h = 112
    for i, (ci, co, s) in enumerate(chans, 1):
        layers.append(dict(name=f"dw{i}", kind="dw", hin=h, cin=ci, cout=ci, stride=s))
        h //= s
        layers.append(dict(name=f"pw{i}", kind="pw", hin=h, cin=ci, cout=co, stride=1))
    layers.append(dict(name="pool", kind="pool", hin=7, cin=1024, cout=1024, stride=1))
    layers.append(dict(name="fc", kind="fc", hin=1, cin=1024, cout=1000, stride=1))
    return layers


def mobilenet_v1_inputs(batch, sparsity_pct, g=4, seed=0):
    """Random-init MobileNet-v1 with batch-norm already folded into the biases.

    Pointwise layers get a balanced group mask at the given sparsity; the
    first conv, the depthwise layers and the classifier stay dense.  Weights
    are He-normal on the kept fan-in so activations stay O(1) through the
    network; biases are N(0, 0.01^2); the image is U[0,1).
    Returns (x, layers) where every layer dict of mobilenet_v1_shapes() gains
    "w", "bias" and, for pw and fc, "mask" and "g".
    """
    x = uniform01(seed, STREAM_X, batch * 224 * 224 * 3).reshape(batch, 224, 224, 3)
    out = []
    for li, spec in enumerate(mobilenet_v1_shapes(), 1):
        L = dict(spec)
        base = 16 * li
        kind, ci, co = L["kind"], L["cin"], L["cout"]
        if kind == "pool":
            out.append(L)
            continue
        L["bias"] = normal(seed, base + STREAM_BIAS, co, 0.01)
        if kind == "conv0":
            L["w"] = normal(seed, base + STREAM_W, co * 27, math.sqrt(2.0 / 27)).reshape(co, 3, 3, ci)
        elif kind == "dw":
            L["w"] = normal(seed, base + STREAM_W, 9 * ci, math.sqrt(2.0 / 9)).reshape(3, 3, ci)
        elif kind == "pw":
            um = _masks.group_mask_balanced(seed, base + STREAM_MASK, co // g, ci, sparsity_pct)
            kept = np.maximum(um.sum(axis=1), 1)
            sig = np.repeat(np.sqrt(2.0 / kept), g).astype(np.float64)
            z = normal(seed, base + STREAM_W, co * ci, 1.0).reshape(co, ci).astype(np.float64)
            L["w"] = (z * sig[:, None]).astype(np.float32).reshape(co, 1, 1, ci)
            L["mask"] = _masks.expand_mask(um, g, 1, 1)
            L["g"] = g
        elif kind == "fc":
            L["w"] = normal(seed, base + STREAM_W, co * ci, math.sqrt(1.0 / ci)).reshape(co, 1, 1, ci)
            L["mask"] = np.ones((co, 1, 1, ci), dtype=np.uint8)
            L["g"] = 4
        out.append(L)
    return x, out
