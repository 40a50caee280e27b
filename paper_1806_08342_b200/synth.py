"""Seeded synthetic inputs for the quantized-convolution workloads.

This module only draws numbers and lists layer shapes; it holds none of the
method's arithmetic (no quantizer, no convolution, no rescaling), so that the
CUDA library and the CPU oracle can both be fed from it without sharing code.

Every array comes from a counter-based Philox generator keyed by
``(seed, stream)``: the same key gives the same array on every machine, and
arrays of different tensors never overlap.

The shapes follow the CNN workloads the whitepaper evaluates (Section 3.1.3:
MobileNet-v1/v2, ResNet-v1-50); the values are random because neither ImageNet
nor trained checkpoints are needed to exercise integer inference.
"""
from __future__ import annotations

import numpy as np


def rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


# --------------------------------------------------------------------------- #
# Single quantized 3x3 convolution (the small correctness workload)
# --------------------------------------------------------------------------- #
def single_conv(seed: int = 1, batch: int = 1, hw: int = 32, c: int = 16, n: int = 32,
                k: int = 3):
    """Float tensors of one conv layer: NHWC input ~U[0,6]; OHWI weights ~N(0, 2/fan_in)
    times a per-output-channel gain that is log-uniform in [0.1, 10] (the dynamic-range
    spread batch-norm folding produces, Section 3.1.2); bias ~N(0, 0.1)."""
    fan_in = k * k * c
    x = rng(seed, 0).uniform(0.0, 6.0, size=(batch, hw, hw, c)).astype(np.float32)
    w = rng(seed, 1).normal(0.0, np.sqrt(2.0 / fan_in), size=(n, k, k, c))
    gain = np.exp(rng(seed, 2).uniform(np.log(0.1), np.log(10.0), size=(n, 1, 1, 1)))
    w = (w * gain).astype(np.float32)
    bias = rng(seed, 3).normal(0.0, 0.1, size=(n,)).astype(np.float32)
    return {"x": x, "w": w, "bias": bias}


# --------------------------------------------------------------------------- #
# Quantized GEMM: uint8 A (MxK), uint8 B (KxN), both asymmetric per layer
# --------------------------------------------------------------------------- #
GEMM_SIZES = (512, 1024, 2048, 4096, 8192)


def gemm_u8(m: int, n: int, k: int, seed: int = 2):
    """Codes uniform over 0..255, zero points uniform in [0,255], int32 bias uniform in
    [-2^15, 2^15].  B is returned K x N row-major, as the workload states it."""
    a = rng(seed, 10).integers(0, 256, size=(m, k), dtype=np.uint8)
    b = rng(seed, 11).integers(0, 256, size=(k, n), dtype=np.uint8)
    z = rng(seed, 12).integers(0, 256, size=2)
    bias = rng(seed, 13).integers(-(1 << 15), (1 << 15) + 1, size=(n,), dtype=np.int32)
    return {"a": a, "b": b, "z_a": int(z[0]), "z_b": int(z[1]), "bias": bias}


def uniform_u8(shape, seed: int, stream: int):
    return rng(seed, stream).integers(0, 256, size=shape, dtype=np.uint8)


def uniform_s8(shape, seed: int, stream: int, lo: int = -127, hi: int = 127):
    return rng(seed, stream).integers(lo, hi + 1, size=shape, dtype=np.int8)


def normal_f32(shape, seed: int, stream: int, std: float = 1.0, mean: float = 0.0):
    return rng(seed, stream).normal(mean, std, size=shape).astype(np.float32)


def uniform_f32(shape, seed: int, stream: int, lo: float = 0.0, hi: float = 1.0):
    return rng(seed, stream).uniform(lo, hi, size=shape).astype(np.float32)


def batchnorm_params(n: int, seed: int, stream: int):
    """gamma~U[0.5,1.5], beta~N(0,0.1), mean~N(0,0.1), var~U[0.5,1.5]."""
    g = rng(seed, stream)
    return {"gamma": g.uniform(0.5, 1.5, n).astype(np.float32),
            "beta": g.normal(0.0, 0.1, n).astype(np.float32),
            "mean": g.normal(0.0, 0.1, n).astype(np.float32),
            "var": g.uniform(0.5, 1.5, n).astype(np.float32)}


# --------------------------------------------------------------------------- #
# Network shapes (Section 3.1.3: MobileNet-v1 / v2, ResNet-v1-50).  Only layer
# geometry and random float parameters live here; how a layer is quantized and
# executed is up to the caller.
#
# A network is a list of ops over named tensors:
#   conv    : src, dst, cin, cout, k, stride, pad, depthwise, act (0 none, 1 ReLU, 2 ReLU6)
#   add     : a, b, dst, act
#   maxpool : src, dst, k, stride, pad
#   avgpool : src, dst            (global)
#   fc      : src, dst, cin, cout (1x1 conv on the pooled vector, int32 logits)
# --------------------------------------------------------------------------- #
def _conv(ops, src, dst, cin, cout, k, stride, act, depthwise=False):
    ops.append({"op": "conv", "src": src, "dst": dst, "cin": cin, "cout": cout, "k": k, "stride": stride,
                "pad": k // 2, "depthwise": depthwise, "act": act})


def mobilenet_v1(classes=1000):
    ops = []
    _conv(ops, "in", "t0", 3, 32, 3, 2, 2)
    widths = [64, 128, 128, 256, 256, 512, 512, 512, 512, 512, 512, 1024, 1024]
    strides = [1, 2, 1, 2, 1, 2, 1, 1, 1, 1, 1, 2, 1]
    c, t = 32, "t0"
    for i, (wd, st) in enumerate(zip(widths, strides)):
        _conv(ops, t, f"dw{i + 1}", c, c, 3, st, 2, depthwise=True)
        _conv(ops, f"dw{i + 1}", f"pw{i + 1}", c, wd, 1, 1, 2)
        c, t = wd, f"pw{i + 1}"
    ops.append({"op": "avgpool", "src": t, "dst": "pool"})
    ops.append({"op": "fc", "src": "pool", "dst": "logits", "cin": c, "cout": classes})
    return ops


def resnet50(classes=1000):
    ops = []
    _conv(ops, "in", "stem", 3, 64, 7, 2, 1)
    ops.append({"op": "maxpool", "src": "stem", "dst": "p0", "k": 3, "stride": 2, "pad": 1})
    c, t = 64, "p0"
    for si, (mid, blocks, stride) in enumerate([(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)]):
        for bi in range(blocks):
            st = stride if bi == 0 else 1          # stride sits on the first 1x1 of a stage (v1)
            n = f"s{si + 2}b{bi + 1}"
            _conv(ops, t, n + "_a", c, mid, 1, st, 1)
            _conv(ops, n + "_a", n + "_b", mid, mid, 3, 1, 1)
            _conv(ops, n + "_b", n + "_c", mid, 4 * mid, 1, 1, 0)
            short = t
            if bi == 0:
                _conv(ops, t, n + "_sc", c, 4 * mid, 1, st, 0)
                short = n + "_sc"
            ops.append({"op": "add", "a": n + "_c", "b": short, "dst": n, "act": 1})
            c, t = 4 * mid, n
    ops.append({"op": "avgpool", "src": t, "dst": "pool"})
    ops.append({"op": "fc", "src": "pool", "dst": "logits", "cin": c, "cout": classes})
    return ops


def mobilenet_v2_14(classes=1000):
    """Width multiplier 1.4, channels rounded to multiples of 8."""
    ops = []
    _conv(ops, "in", "stem", 3, 48, 3, 2, 2)
    c, t = 48, "stem"
    cfg = [(1, 24, 1, 1), (6, 32, 2, 2), (6, 48, 3, 2), (6, 88, 4, 2), (6, 136, 3, 1), (6, 224, 3, 2), (6, 448, 1, 1)]
    bi = 0
    for expand, cout, reps, stride in cfg:
        for r in range(reps):
            bi += 1
            st = stride if r == 0 else 1
            n, e, src = f"b{bi}", c * expand, t
            if expand != 1:
                _conv(ops, src, n + "_e", c, e, 1, 1, 2)
                src = n + "_e"
            _conv(ops, src, n + "_d", e, e, 3, st, 2, depthwise=True)
            _conv(ops, n + "_d", n + "_p", e, cout, 1, 1, 0)            # linear bottleneck
            if st == 1 and c == cout:
                ops.append({"op": "add", "a": n + "_p", "b": t, "dst": n, "act": 0})
                t = n
            else:
                t = n + "_p"
            c = cout
    _conv(ops, t, "last", c, 1792, 1, 1, 2)
    ops.append({"op": "avgpool", "src": "last", "dst": "pool"})
    ops.append({"op": "fc", "src": "pool", "dst": "logits", "cin": 1792, "cout": classes})
    return ops


NETWORKS = {"mobilenet_v1": mobilenet_v1, "resnet50": resnet50, "mobilenet_v2_14": mobilenet_v2_14}


def network_input(batch, resolution, seed):
    """uint8 images, uniform over 0..255 (read as real values in [0,1]: scale 1/255, zero point 0)."""
    return uniform_u8((batch, resolution, resolution, 3), seed, 500)


def layer_params(op, index, seed):
    """Float parameters of conv / fc op number `index`: He-normal weights (OHWI; depthwise: HWC),
    batch-norm statistics (conv) or a small bias (fc)."""
    if op["op"] == "fc":
        w = normal_f32((op["cout"], 1, 1, op["cin"]), seed, 1000 + 4 * index, std=np.sqrt(1.0 / op["cin"]))
        return {"w": w, "bias": normal_f32((op["cout"],), seed, 1001 + 4 * index, std=0.05)}
    k = op["k"]
    if op["depthwise"]:
        w = normal_f32((k, k, op["cin"]), seed, 1000 + 4 * index, std=np.sqrt(2.0 / (k * k)))
    else:
        w = normal_f32((op["cout"], k, k, op["cin"]), seed, 1000 + 4 * index, std=np.sqrt(2.0 / (k * k * op["cin"])))
    return {"w": w, "bn": batchnorm_params(op["cout"], seed, 1002 + 4 * index)}
