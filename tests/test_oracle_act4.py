"""Pins of the oracle's 4-bit activation pieces (Section 3.2.4, Table 6: 4-bit activations).

Expected values come from the definitions, not from the functions under test: the byte layout is
written out by hand for all 256 byte values, the clamp of a fused activation is checked against real
arithmetic (the code of real 0 and of real 6), and a whole 4-bit layer -- quantize, integer
convolution, requantize to 4 bits -- is compared with a float64 convolution of the dequantized
tensors, whose accumulators must match exactly and whose outputs must sit within half a step."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_1806_08342_b200 import synth


def test_u4_layout_for_every_byte_value():
    # byte b holds element 2i = b & 15 (low nibble) and element 2i + 1 = b >> 4 (high nibble)
    codes = np.array([[b & 15, b >> 4] for b in range(256)], np.uint8).reshape(1, 512)
    packed = oracle.pack_u4(codes)
    assert packed.shape == (1, 256) and np.array_equal(packed[0], np.arange(256, dtype=np.uint8))
    assert np.array_equal(oracle.unpack_u4(packed, 512), codes)
    # an odd tail leaves the high nibble zero; rows keep their pitch
    odd = np.array([[1, 2, 3], [15, 0, 9]], np.uint8)
    p = oracle.pack_u4(odd, packed_pitch=4)
    assert p.tolist() == [[0x21, 0x03, 0, 0], [0x0F, 0x09, 0, 0]]
    assert np.array_equal(oracle.unpack_u4(p, 3), odd)
    with pytest.raises(oracle.OracleError):
        oracle.pack_u4(np.array([[16, 0]], np.uint8))


def test_activation_clamp_for_any_width_matches_real_arithmetic():
    g = synth.rng(91, 0)
    for _ in range(500):
        bits = int(g.integers(2, 9))
        top = (1 << bits) - 1
        lo, hi = -float(g.uniform(0, 3)), float(g.uniform(0.5, 9))
        p = oracle.affine_params(np.float32(lo), np.float32(hi), bits)
        s, z = Fraction(float(p["scale"])), int(p["zero_point"])
        assert oracle.activation_range_bits(0, p["scale"], z, bits) == (0, top)
        assert oracle.activation_range_bits(1, p["scale"], z, bits) == (z, top)
        amin, amax = oracle.activation_range_bits(2, p["scale"], z, bits)
        assert amin == z and amax <= top
        if amax < top:                                   # the code whose real value is nearest to 6
            assert abs((amax - z) * s - 6) <= s / 2
        else:                                            # 6 lies at or beyond the top code
            assert (top - z) * s <= 6 + s / 2
    for kind in (0, 1, 2):                               # at 8 bits it is the 8-bit rule
        assert oracle.activation_range_bits(kind, 0.0235, 3, 8) == oracle.activation_range(kind, 0.0235, 3)


def test_four_bit_activation_layer_against_float64():
    """4-bit activations in and out, 8-bit per-channel weights (a row of Table 6)."""
    g = synth.rng(92, 0)
    x = g.uniform(-1.0, 5.0, size=(2, 9, 9, 8)).astype(np.float32)
    w = g.normal(0, 0.2, size=(6, 3, 3, 8)).astype(np.float32)
    xp = oracle.affine_params(x.min(), x.max(), 4)
    assert 0 <= xp["zero_point"] <= 15
    xq = oracle.quantize(x, xp, None, 0, 15)
    assert xq.min() >= 0 and xq.max() == 15 and len(np.unique(xq)) == 16
    # storage round trip
    xq8 = xq.astype(np.uint8)
    assert np.array_equal(oracle.unpack_u4(oracle.pack_u4(xq8), 8), xq8)
    wp = oracle.calibrate_minmax(w, 0, 8, True)
    wq = oracle.quantize(w, wp, 0, -127, 127)
    zx = int(xp["zero_point"])
    acc = oracle.conv2d_acc(xq8, zx, wq, None, None, 1, 1)
    # float64 convolution of the dequantized tensors, zero padded in the real domain
    xr = (xq.astype(np.float64) - zx)
    pad = np.zeros((2, 11, 11, 8))
    pad[:, 1:10, 1:10] = xr
    ref = np.zeros((2, 9, 9, 6))
    for i in range(3):
        for j in range(3):
            ref += pad[:, i:i + 9, j:j + 9] @ wq[:, i, j, :].astype(np.float64).T
    assert np.array_equal(acc, ref.astype(np.int64))
    # requantize to a 4-bit output with ReLU: every output within half a step of the real value
    real = ref * float(xp["scale"]) * wp["scale"].astype(np.float64)
    yp = oracle.affine_params(np.float32(0.0), np.float32(real.max()), 4)
    amin, amax = oracle.activation_range_bits(1, yp["scale"], int(yp["zero_point"]), 4)
    mr = [oracle.quantize_multiplier(float(xp["scale"]) * float(s) / float(yp["scale"])) for s in wp["scale"]]
    y = oracle.requantize(acc, np.array([m for m, _ in mr], np.int32), np.array([r for _, r in mr], np.int32),
                          int(yp["zero_point"]), amin, amax)
    assert y.min() >= 0 and y.max() <= 15
    back = (y - int(yp["zero_point"])) * float(yp["scale"])
    want = np.clip(real, 0.0, (15 - int(yp["zero_point"])) * float(yp["scale"]))
    assert np.abs(back - want).max() <= 0.5 * float(yp["scale"]) * (1 + 1e-6)
