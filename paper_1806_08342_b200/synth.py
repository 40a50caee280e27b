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
