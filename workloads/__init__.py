"""Seeded synthetic inputs: quantized network parameter sets and uint8 images.

This module only produces INPUTS (layer lists with random int8 weights and
requantisation parameters, random images).  It holds none of the method's
arithmetic and is the one module that both the CPU oracle's tests and the CUDA
library's callers may import.

The networks have the shapes of the paper's workloads (Sec. 4.1 "Implementation
Details": ResNet-20 on 3x32x32 CIFAR-10 images, ResNet-50 on 3x224x224
Caltech-101 images with 101 classes) plus a deeper CIFAR-shaped ResNet-110 and
a tiny CNN; weights are random because the trained checkpoints and the data
sets are not available.  Images are uniform random bytes.

A model is ``{"name", "in_shape": (C, H, W), "n_classes", "layers": [dict]}``;
layer ``i`` reads tensor ``in_tensor`` (0 = the network input) and writes
tensor ``i + 1``.
"""
from __future__ import annotations

import numpy as np

OP_CONV2D, OP_FC, OP_GAVGPOOL, OP_MAXPOOL = 0, 1, 2, 3

_GAMMA = np.uint64(0x9E3779B97F4A7C15)


class SplitMix64:
    """Vectorised SplitMix64 stream (Steele, Lea, Flood 2014)."""

    def __init__(self, seed: int):
        self.seed = np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
        self.pos = 0

    def raw(self, n: int) -> np.ndarray:
        with np.errstate(over="ignore"):
            idx = np.arange(self.pos + 1, self.pos + n + 1, dtype=np.uint64)
            z = self.seed + idx * _GAMMA
            z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
            z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
            z = z ^ (z >> np.uint64(31))
        self.pos += n
        return z

    def ints(self, n: int, lo: int, hi: int) -> np.ndarray:
        """n integers uniform in [lo, hi] (int64)."""
        span = np.uint64(hi - lo + 1)
        top = self.raw(n) >> np.uint64(32)
        return (np.int64(lo) + ((top * span) >> np.uint64(32)).astype(np.int64))


def _conv(rng, in_tensor, cin, cout, k, stride, pad, relu, zp_in, zp_out,
          res_tensor=-1, zp_res=0, op=OP_CONV2D):
    n_w = cout * cin * k * k
    layer = dict(op=op, in_tensor=in_tensor, res_tensor=res_tensor, cin=cin, cout=cout,
                 kh=k, kw=k, stride=stride, pad=pad, relu=int(relu),
                 zp_in=zp_in, zp_out=zp_out, zp_res=zp_res,
                 w=rng.ints(n_w, -127, 127).astype(np.int8).reshape(cout, cin, k, k),
                 bias=rng.ints(cout, -(1 << 12), 1 << 12).astype(np.int32),
                 mult=rng.ints(cout, 1 << 30, (1 << 31) - 1).astype(np.int32),
                 shift=rng.ints(cout, 8, 12).astype(np.int8),
                 res_mult=0, res_shift=0)
    if res_tensor >= 0:
        layer["res_mult"] = int(rng.ints(1, 1 << 30, (1 << 31) - 1)[0])
    return layer


def _gavgpool(in_tensor, c, hw, zp):
    """Average over hw pixels as a fixed-point multiplier: mult / 2^(31+shift) ~ 1/hw."""
    shift = 0
    while (1 << (shift + 1)) <= hw:          # largest shift with 2^shift <= hw
        shift += 1
    # mult in [2^30, 2^31): 1/hw = mult / 2^(31 + s)  with  s = shift - 1 (+1 if hw not a power of two)
    if (1 << shift) == hw:
        s, mult = shift - 1, 1 << 30
    else:
        s = shift
        mult = int(round((1 << (31 + s)) / hw))
    return dict(op=OP_GAVGPOOL, in_tensor=in_tensor, res_tensor=-1, cin=c, cout=c, kh=1, kw=1,
                stride=1, pad=0, relu=0, zp_in=zp, zp_out=zp, zp_res=0, w=None, bias=None,
                mult=np.array([mult], dtype=np.int32), shift=np.array([s], dtype=np.int8),
                res_mult=0, res_shift=0)


def _maxpool(in_tensor, c, k, stride, pad, zp):
    return dict(op=OP_MAXPOOL, in_tensor=in_tensor, res_tensor=-1, cin=c, cout=c, kh=k, kw=k,
                stride=stride, pad=pad, relu=0, zp_in=zp, zp_out=zp, zp_res=0, w=None, bias=None,
                mult=np.array([1 << 30], dtype=np.int32), shift=np.array([0], dtype=np.int8),
                res_mult=0, res_shift=0)


RELU_ZP = -128   # zero-point of every ReLU output: the ReLU is the lower clamp


def tiny_cnn(seed: int = 0x15170000) -> dict:
    """conv3x3 3->16 ReLU; conv3x3 16->32 stride 2 ReLU; global avg-pool; FC 32->10."""
    rng = SplitMix64(seed)
    L = [_conv(rng, 0, 3, 16, 3, 1, 1, True, 0, RELU_ZP),
         _conv(rng, 1, 16, 32, 3, 2, 1, True, RELU_ZP, RELU_ZP),
         _gavgpool(2, 32, 16 * 16, RELU_ZP),
         _conv(rng, 3, 32, 10, 1, 1, 0, False, RELU_ZP, 0, op=OP_FC)]
    return dict(name="tiny_cnn", in_shape=(3, 32, 32), n_classes=10, layers=L)


def cifar_resnet(blocks_per_stage: int, seed: int, n_classes: int = 10, hw: int = 32,
                 widths=(16, 32, 64)) -> dict:
    """CIFAR-style ResNet of 6*blocks_per_stage+2 layers: 3 stages of basic blocks,
    1x1 stride-2 projection shortcuts at the two stage transitions, integer residual adds."""
    rng = SplitMix64(seed)
    L = [_conv(rng, 0, 3, widths[0], 3, 1, 1, True, 0, RELU_ZP)]
    cur, cin, size = 1, widths[0], hw
    for si, width in enumerate(widths):
        for b in range(blocks_per_stage):
            stride = 2 if (si > 0 and b == 0) else 1
            L.append(_conv(rng, cur, cin, width, 3, stride, 1, True, RELU_ZP, RELU_ZP))
            y1 = len(L)
            if stride != 1 or cin != width:
                L.append(_conv(rng, cur, cin, width, 1, stride, 0, False, RELU_ZP, 0))
                short, zp_short = len(L), 0
            else:
                short, zp_short = cur, RELU_ZP
            L.append(_conv(rng, y1, width, width, 3, 1, 1, True, RELU_ZP, RELU_ZP,
                           res_tensor=short, zp_res=zp_short))
            cur, cin = len(L), width
            size //= stride
    L.append(_gavgpool(cur, cin, size * size, RELU_ZP))
    L.append(_conv(rng, len(L), cin, n_classes, 1, 1, 0, False, RELU_ZP, 0, op=OP_FC))
    return dict(name=f"resnet{6 * blocks_per_stage + 2}", in_shape=(3, hw, hw),
                n_classes=n_classes, layers=L)


def resnet20(seed: int = 0x15170001) -> dict:
    return cifar_resnet(3, seed)


def resnet110(seed: int = 0x15170002) -> dict:
    return cifar_resnet(18, seed)


def resnet50(seed: int = 0x15170003, n_classes: int = 101, hw: int = 224,
             blocks=(3, 4, 6, 3), base: int = 64) -> dict:
    """Bottleneck ResNet (stride on the 3x3), 7x7 stride-2 stem, 3x3 stride-2 max-pool."""
    rng = SplitMix64(seed)
    L = [_conv(rng, 0, 3, base, 7, 2, 3, True, 0, RELU_ZP)]
    size = (hw + 6 - 7) // 2 + 1
    L.append(_maxpool(1, base, 3, 2, 1, RELU_ZP))
    size = (size + 2 - 3) // 2 + 1
    cur, cin = 2, base
    for si, nb in enumerate(blocks):
        mid = base << si
        out = mid * 4
        for b in range(nb):
            stride = 2 if (si > 0 and b == 0) else 1
            L.append(_conv(rng, cur, cin, mid, 1, 1, 0, True, RELU_ZP, RELU_ZP))
            L.append(_conv(rng, len(L), mid, mid, 3, stride, 1, True, RELU_ZP, RELU_ZP))
            y2 = len(L)
            if b == 0:
                L.append(_conv(rng, cur, cin, out, 1, stride, 0, False, RELU_ZP, 0))
                short, zp_short = len(L), 0
            else:
                short, zp_short = cur, RELU_ZP
            L.append(_conv(rng, y2, mid, out, 1, 1, 0, True, RELU_ZP, RELU_ZP,
                           res_tensor=short, zp_res=zp_short))
            cur, cin = len(L), out
            size //= stride
    L.append(_gavgpool(cur, cin, size * size, RELU_ZP))
    L.append(_conv(rng, len(L), cin, n_classes, 1, 1, 0, False, RELU_ZP, 0, op=OP_FC))
    return dict(name="resnet50", in_shape=(3, hw, hw), n_classes=n_classes, layers=L)


def images(n: int, shape=(3, 32, 32), seed: int = 0x15171000) -> np.ndarray:
    """n images of uniform random bytes, CHW, uint8."""
    rng = SplitMix64(seed)
    c, h, w = shape
    return rng.ints(n * c * h * w, 0, 255).astype(np.uint8).reshape(n, c, h, w)


def macs_per_sample(model: dict) -> int:
    """Multiply-accumulates of one forward pass (true, unpadded shapes)."""
    c, h, w = model["in_shape"]
    shapes = [(c, h, w)]
    total = 0
    for L in model["layers"]:
        ci, hi, wi = shapes[L["in_tensor"]]
        if L["op"] == OP_CONV2D:
            ho = (hi + 2 * L["pad"] - L["kh"]) // L["stride"] + 1
            wo = (wi + 2 * L["pad"] - L["kw"]) // L["stride"] + 1
            total += ho * wo * L["cout"] * ci * L["kh"] * L["kw"]
            shapes.append((L["cout"], ho, wo))
        elif L["op"] == OP_FC:
            total += L["cout"] * ci
            shapes.append((L["cout"], 1, 1))
        elif L["op"] == OP_GAVGPOOL:
            shapes.append((ci, 1, 1))
        else:
            ho = (hi + 2 * L["pad"] - L["kh"]) // L["stride"] + 1
            wo = (wi + 2 * L["pad"] - L["kw"]) // L["stride"] + 1
            shapes.append((ci, ho, wo))
    return total


# The five benchmark configurations (seeds: model 0x15170000+cfg, images 0x15171000+cfg).
NOISE_SEED = 2021

CONFIGS = {
    0: dict(model=lambda: tiny_cnn(0x15170000), n_images=1, shape=(3, 32, 32),
            sigmas=(0.25,), N0=100, N=1000, alpha=0.001, image_seed=0x15171000),
    1: dict(model=lambda: cifar_resnet(3, 0x15170001), n_images=100, shape=(3, 32, 32),
            sigmas=(0.12, 0.25, 0.5), N0=100, N=100000, alpha=0.001, image_seed=0x15171001),
    2: dict(model=lambda: cifar_resnet(18, 0x15170002), n_images=500, shape=(3, 32, 32),
            sigmas=(0.25,), N0=100, N=100000, alpha=0.001, image_seed=0x15171002),
    3: dict(model=lambda: resnet50(0x15170003), n_images=50, shape=(3, 224, 224),
            sigmas=(0.5,), N0=100, N=10000, alpha=0.001, image_seed=0x15171003),
    4: dict(model=lambda: cifar_resnet(18, 0x15170002), n_images=20, shape=(3, 32, 32),
            sigmas=(0.12, 0.25, 0.5, 1.0), N0=100, N=100000, alpha=0.001,
            image_seed=0x15171004, batches=(256, 1024, 4096, 16384)),
}


# ---------------------------------------------------------------------------------------------
# Test models whose votes spread over several classes.
#
# A network with random weights puts (almost) every noisy copy of an image in one class, which
# leaves vote histograms, tie-breaking, ABSTAIN and non-maximal radii unexercised.  The variant
# below swaps the final FC layer for one with small weights, one multiplier/shift for all
# classes and a caller-supplied bias vector.  With biases that cancel each class's mean
# accumulator on one chosen image (``spread_bias.json``, written by ``calibrate_spread.py``
# beside this file from pooled features the CPU oracle reports), the logits of that image's
# noisy copies differ by a few units only: votes spread and exact ties for the maximum occur.
SPREAD_IMAGE_SEED = 0x15172000


def with_spread_head(model: dict, bias, seed: int = 0x15173000, delta: int = 4, shift: int = 6) -> dict:
    rng = SplitMix64(seed)
    fc = dict(model["layers"][-1])
    cout, cin = fc["cout"], fc["cin"]
    fc["w"] = rng.ints(cout * cin, -delta, delta).astype(np.int8).reshape(cout, cin, 1, 1)
    fc["mult"] = np.full(cout, int(rng.ints(1, 1 << 30, (1 << 31) - 1)[0]), dtype=np.int32)
    fc["shift"] = np.full(cout, shift, dtype=np.int8)
    fc["bias"] = np.asarray(bias, dtype=np.int32).reshape(cout)
    return dict(model, name=model["name"] + "_spread", layers=list(model["layers"][:-1]) + [fc])


def spread_image(shape=(3, 32, 32)) -> np.ndarray:
    """The image the stored biases were balanced on."""
    return images(1, shape=shape, seed=SPREAD_IMAGE_SEED)[0]


# (delta, shift) of the head per base network: the tiny CNN's pooled features move less under noise
SPREAD_HEADS = {"tiny_cnn": (16, 4), "resnet20": (4, 6), "resnet110": (4, 6)}


def spread_base(name: str) -> dict:
    return {"tiny_cnn": tiny_cnn, "resnet20": resnet20, "resnet110": resnet110}[name]()


def spread_model(name: str, boost: int = 0) -> dict:
    """tiny_cnn / resnet20 / resnet110 with the spread-vote head and its stored biases; `boost` is added to
    class 0's bias (a favourite class: a majority that is not unanimous)."""
    import json
    import os
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "spread_bias.json")) as f:
        bias = list(json.load(f)[name])
    bias[0] += boost
    delta, shift = SPREAD_HEADS[name]
    return with_spread_head(spread_base(name), bias, delta=delta, shift=shift)
