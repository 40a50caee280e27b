"""Pins for the oracle's convolution, requantisation, BN folding and glue ops.

Expected values come from float64 / exact-rational restatements of the paper's
definitions and from library routines (numpy matmul, sliding windows), never from
the oracle functions themselves.
"""
from fractions import Fraction

import numpy as np
import pytest
from numpy.lib.stride_tricks import sliding_window_view

import oracle


def conv_f64(x, w, stride, pad):
    """Textbook float64 cross-correlation, NHWC x OHWI, zero padding."""
    xp = np.pad(x, ((0, 0), (pad, pad), (pad, pad), (0, 0)))
    kh, kw = w.shape[1:3]
    win = sliding_window_view(xp, (kh, kw), axis=(1, 2))[:, ::stride, ::stride]
    return np.einsum("bhwcij,oijc->bhwo", win, w, optimize=True)   # win: B,OH,OW,C,kh,kw


def rand_case(g, b, h, w, c, n, k, signed_w=True, pitch=None):
    pitch = pitch or c
    x = g.integers(0, 256, size=(b, h, w, pitch), dtype=np.uint8)
    if signed_w:
        wq = g.integers(-127, 128, size=(n, k, k, c)).astype(np.int32)
    else:
        wq = g.integers(0, 256, size=(n, k, k, c)).astype(np.int32)
    bias = g.integers(-5000, 5000, size=n).astype(np.int32)
    return x, wq, bias


@pytest.mark.parametrize("stride,pad,k", [(1, 1, 3), (2, 1, 3), (1, 0, 1), (2, 0, 1), (2, 3, 7)])
def test_accumulators_equal_float64_conv_of_dequantized(stride, pad, k):
    # Eq. 4: y = Dw Dx conv(wQ - zw, xQ - zx).  Dequantize both tensors (Eq. 3), convolve in
    # float64, divide by Dw[n] Dx: every value is an integer far below 2^53, so the int32
    # accumulator must match exactly.
    g = np.random.default_rng(100 + k + stride)
    b, h, w, c, n = 2, 9, 8, 5, 4
    x, wq, bias = rand_case(g, b, h, w, c, n, k, signed_w=False, pitch=8)
    z_x = 117
    z_w = g.integers(0, 256, size=n).astype(np.int32)
    dx = 0.0235
    dw = g.uniform(0.001, 0.1, size=n)
    xf = (x[..., :c].astype(np.float64) - z_x) * dx
    wf = (wq.astype(np.float64) - z_w[:, None, None, None]) * dw[:, None, None, None]
    want = conv_f64(xf, wf, stride, pad) / (dx * dw) + bias
    got = oracle.conv2d_acc(x, z_x, wq, z_w, bias, stride, pad, c=c)
    assert got.shape == want.shape
    assert np.array_equal(got, np.rint(want).astype(np.int64))
    assert np.abs(want - np.rint(want)).max() < 1e-3


def test_zero_zero_points_reduce_to_integer_convolution():
    g = np.random.default_rng(5)
    x, wq, _ = rand_case(g, 1, 6, 7, 3, 5, 3)
    want = conv_f64(x.astype(np.float64), wq.astype(np.float64), 1, 1)
    got = oracle.conv2d_acc(x, 0, wq, None, None, 1, 1)
    assert np.array_equal(got, want.astype(np.int64))


def test_pointwise_on_1x1_image_is_integer_matmul():
    g = np.random.default_rng(6)
    m, k, n = 37, 53, 19
    a = g.integers(0, 256, size=(m, k), dtype=np.uint8)
    bq = g.integers(0, 256, size=(k, n), dtype=np.uint8)
    za, zb = 200, 3
    want = (a.astype(np.int64) - za) @ (bq.astype(np.int64) - zb)
    got = oracle.conv2d_acc(a.reshape(m, 1, 1, k), za, bq.T.reshape(n, 1, 1, k),
                            np.full(n, zb, np.int32), None, 1, 0)
    assert np.array_equal(got.reshape(m, n), want)


def test_zero_padding_is_the_zero_point_code():
    # Section 2.1: zero padding must not cause error -- a padded conv equals the unpadded
    # conv of an image explicitly bordered with the code z_x.
    g = np.random.default_rng(8)
    x, wq, bias = rand_case(g, 2, 7, 6, 4, 3, 3)
    z_x = 91
    xb = np.full((2, 9, 8, 4), z_x, np.uint8)
    xb[:, 1:-1, 1:-1] = x
    a = oracle.conv2d_acc(x, z_x, wq, None, bias, 1, 1)
    b = oracle.conv2d_acc(xb, z_x, wq, None, bias, 1, 0)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("stride,pad,k", [(1, 1, 3), (2, 1, 3), (1, 0, 1)])
def test_expanded_form_equals_defining_form(stride, pad, k):
    # Eq. 5-6 against Eq. 4; fixes the count on the constant term: K_valid * zx * zw.
    g = np.random.default_rng(9)
    x, wq, bias = rand_case(g, 2, 6, 5, 6, 4, k, signed_w=False)
    z_w = np.full(4, 77, np.int32)
    a = oracle.conv2d_acc(x, 133, wq, z_w, bias, stride, pad)
    b = oracle.conv2d_acc(x, 133, wq, z_w, bias, stride, pad, expanded=True)
    assert np.array_equal(a, b)
    # and the expanded form, retyped with numpy for the interior (no padding effects)
    if pad == 0 and k == 1 and stride == 1:
        xi, wi = x.astype(np.int64), wq.astype(np.int64).reshape(4, 6)
        raw = xi @ wi.T
        want = (raw - 77 * xi.sum(-1, keepdims=True) - 133 * wi.sum(-1)[None, None, None, :]
                + 6 * 133 * 77 + bias)
        assert np.array_equal(a, want)


def test_accumulator_overflow_is_reported():
    x = np.full((1, 1, 1, 70000), 255, np.uint8)
    w = np.full((1, 1, 1, 70000), 127, np.int32)
    with pytest.raises(oracle.OracleError):
        oracle.conv2d_acc(x, 0, w, None, None, 1, 0)


def test_depthwise_equals_block_diagonal_conv_and_float64():
    g = np.random.default_rng(12)
    b, h, w, c = 2, 7, 9, 6
    x = g.integers(0, 256, size=(b, h, w, 8), dtype=np.uint8)
    wq = g.integers(-127, 128, size=(3, 3, c)).astype(np.int32)
    bias = g.integers(-300, 300, size=c).astype(np.int32)
    z_x = 19
    for stride in (1, 2):
        got = oracle.depthwise_acc(x, z_x, wq, None, bias, stride, 1, c=c)
        dense = np.zeros((c, 3, 3, c), np.int32)
        for ch in range(c):
            dense[ch, :, :, ch] = wq[:, :, ch]
        assert np.array_equal(got, oracle.conv2d_acc(x, z_x, dense, None, bias, stride, 1, c=c))
        xf = x[..., :c].astype(np.float64) - z_x
        xpad = np.pad(xf, ((0, 0), (1, 1), (1, 1), (0, 0)))
        win = sliding_window_view(xpad, (3, 3), axis=(1, 2))[:, ::stride, ::stride]
        want = np.einsum("bhwcij,ijc->bhwc", win, wq.astype(np.float64)) + bias
        assert np.array_equal(got, want.astype(np.int64))
    # asymmetric depthwise weights (per-channel zero point)
    zw = g.integers(0, 256, size=c).astype(np.int32)
    wu = g.integers(0, 256, size=(3, 3, c)).astype(np.int32)
    got = oracle.depthwise_acc(x, z_x, wu, zw, None, 1, 1, c=c)
    xpad = np.pad(x[..., :c].astype(np.float64) - z_x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    win = sliding_window_view(xpad, (3, 3), axis=(1, 2))
    want = np.einsum("bhwcij,ijc->bhwc", win, wu.astype(np.float64) - zw)
    assert np.array_equal(got, want.astype(np.int64))


# ------------------------------------------------------------------------------------- #
def test_multiplier_precision_and_special_cases():
    g = np.random.default_rng(1)
    for M in list(10 ** g.uniform(-8, 2, 3000)) + [1.0, 0.5, 0.75, 2.0 ** -20, 1 - 2.0 ** -40]:
        m, r = oracle.quantize_multiplier(float(M))
        assert 2 ** 30 <= m < 2 ** 31 and 1 <= r <= 62
        approx = Fraction(m, 2 ** r)
        assert abs(approx / Fraction(float(M)) - 1) <= Fraction(1, 2 ** 31)
    assert oracle.quantize_multiplier(0.0) == (0, 1)
    assert oracle.quantize_multiplier(0.5) == (2 ** 30, 31)
    assert oracle.quantize_multiplier(2.0 ** -7) == (2 ** 30, 37)
    with pytest.raises(oracle.OracleError):
        oracle.quantize_multiplier(2.0 ** 31)
    with pytest.raises(oracle.OracleError):
        oracle.quantize_multiplier(-1.0)


def test_requantize_against_exact_rational():
    g = np.random.default_rng(2)
    n = 16
    M = 10 ** g.uniform(-6, -1, n)
    mr = [oracle.quantize_multiplier(float(v)) for v in M]
    mult = np.array([a for a, _ in mr], np.int32)
    rsh = np.array([b for _, b in mr], np.int32)
    acc = g.integers(-2 ** 31, 2 ** 31, size=(400, n)).astype(np.int32)
    acc[0] = 0
    acc[1] = 2 ** 31 - 1
    acc[2] = -2 ** 31
    zy = 13
    got = oracle.requantize(acc, mult, rsh, zy, -2 ** 31, 2 ** 31 - 1)
    for p in range(acc.shape[0]):
        for c in range(n):
            # exact: zy + floor(acc * m / 2^r + 1/2) in rationals
            v = Fraction(int(acc[p, c]) * int(mult[c]), 2 ** int(rsh[c])) + Fraction(1, 2)
            assert got[p, c] == zy + (v.numerator // v.denominator)
            # and within one code of the real-valued rescale
            assert abs((got[p, c] - zy) - int(acc[p, c]) * M[c]) <= 0.5 + abs(int(acc[p, c])) * M[c] * 2.0 ** -30 + 1e-9
    assert np.all(got[0] == zy)                       # acc = 0 -> y = z_y
    # power-of-two multiplier is an exact rounding shift, ties toward +infinity
    m, r = oracle.quantize_multiplier(2.0 ** -3)
    a = np.array([[12, 4, -4, -12, 7, -7, 20]], np.int32).T
    got = oracle.requantize(a, np.array([m], np.int32), np.array([r], np.int32), 0, -99, 99)
    assert got.ravel().tolist() == [2, 1, 0, -1, 1, -1, 3]
    # clamp
    got = oracle.requantize(a, np.array([m], np.int32), np.array([r], np.int32), 0, 0, 2)
    assert got.ravel().tolist() == [2, 1, 0, 0, 1, 0, 2]


def test_activation_ranges():
    assert oracle.activation_range(0, 0.1, 7) == (0, 255)
    assert oracle.activation_range(1, 0.1, 7) == (7, 255)
    assert oracle.activation_range(2, 6.0 / 255.0, 0) == (0, 255)
    assert oracle.activation_range(2, 0.05, 10) == (10, 130)
    assert oracle.activation_range(2, 0.01, 10) == (10, 255)


def test_batchnorm_fold_identity():
    # Eq. 20-21: conv(x, W_inf) + Bias_inf == gamma (conv(x, W) + b - mu) / sigma + beta
    g = np.random.default_rng(4)
    n, k, c = 6, 3, 5
    w = g.normal(size=(n, k, k, c)).astype(np.float32)
    cb = g.normal(size=n).astype(np.float32)
    gamma = g.uniform(0.5, 1.5, n).astype(np.float32)
    beta = g.normal(size=n).astype(np.float32)
    mean = g.normal(size=n).astype(np.float32)
    var = g.uniform(0.5, 1.5, n).astype(np.float32)
    eps = 1e-3
    x = g.normal(size=(2, 6, 6, c))
    for bias in (cb, None):
        w_inf, b_inf = oracle.fold_batchnorm(w, bias, gamma, beta, mean, var, eps)
        sigma = np.sqrt(var.astype(np.float64) + np.float64(np.float32(eps)))
        pre = conv_f64(x, w.astype(np.float64), 1, 1) + (0 if bias is None else bias)
        want = gamma * (pre - mean) / sigma + beta
        got = conv_f64(x, w_inf.astype(np.float64), 1, 1) + b_inf
        assert np.allclose(got, want, rtol=0, atol=2e-5)       # fp32 rounding of W_inf, b_inf
        assert np.allclose(w_inf, gamma[:, None, None, None] * w / sigma[:, None, None, None],
                           rtol=1e-7, atol=0)
    # gamma = sigma, beta = mu = 0 is the identity
    one = np.ones(n, np.float32)
    zero = np.zeros(n, np.float32)
    w_inf, b_inf = oracle.fold_batchnorm(w, None, one, zero, zero, one, 0.0)
    assert np.array_equal(w_inf, w) and np.array_equal(b_inf, zero)


def test_bias_quantization():
    bias = np.array([0.1, -0.2, 0.0, 1e9], np.float32)
    ws = np.array([0.01, 0.02, 0.5, 1e-6], np.float32)
    got = oracle.quantize_bias(bias, 0.05, ws)
    s = np.float64(np.float32(0.05)) * ws.astype(np.float64)
    want = np.clip(np.rint(bias.astype(np.float64) / s), -2 ** 31, 2 ** 31 - 1)
    assert got.tolist() == want.astype(np.int64).tolist()
    assert got[3] == 2 ** 31 - 1


# ------------------------------------------------------------------------------------- #
def test_add_rescale():
    g = np.random.default_rng(14)
    a = g.integers(0, 256, size=(50, 8), dtype=np.uint8)
    b = g.integers(0, 256, size=(50, 8), dtype=np.uint8)
    # equal scales: exact saturating integer add of the zero-point-free codes
    ma, mb, r = oracle.add_params(0.1, 0.1, 0.1)
    assert (ma, mb, r) == (2 ** 30, 2 ** 30, 30)
    y = oracle.add_u8(a, 10, ma, b, 20, mb, r, 5, 0, 255)
    want = np.clip(a.astype(int) - 10 + b.astype(int) - 20 + 5, 0, 255)
    assert np.array_equal(y, want)
    # general scales: exact rational of the stated formula, and <= 1 code from the real sum
    sa, sb, sy = 0.043, 0.11, 0.13
    ma, mb, r = oracle.add_params(sa, sb, sy)
    Ma = float(np.float32(sa)) / float(np.float32(sy))
    Mb = float(np.float32(sb)) / float(np.float32(sy))
    assert abs(Fraction(mb, 2 ** r) / Fraction(Mb) - 1) <= Fraction(1, 2 ** 31)
    assert abs(ma - Ma * 2 ** r) <= 0.5
    y = oracle.add_u8(a, 3, ma, b, 200, mb, r, 100, 100, 255, c=6)   # fused ReLU clamp
    for i in range(50):
        for ch in range(6):
            v = Fraction((int(a[i, ch]) - 3) * ma + (int(b[i, ch]) - 200) * mb, 2 ** r) + Fraction(1, 2)
            exact = min(max(100 + v.numerator // v.denominator, 100), 255)
            assert y[i, ch] == exact
            real = 100 + (int(a[i, ch]) - 3) * Ma + (int(b[i, ch]) - 200) * Mb
            assert abs(y[i, ch] - min(max(real, 100), 255)) <= 0.5 + 1e-3
    assert np.all(y[:, 6:] == 0)


def test_maxpool_is_max_of_dequantized_values():
    g = np.random.default_rng(15)
    x = g.integers(0, 256, size=(2, 9, 9, 4), dtype=np.uint8)
    y = oracle.maxpool_u8(x, 3, 2, 1)
    assert y.shape == (2, 5, 5, 4)
    d, z = 0.05, 30
    xf = (x.astype(np.float64) - z) * d
    xp = np.pad(xf, ((0, 0), (1, 1), (1, 1), (0, 0)), constant_values=-np.inf)
    win = sliding_window_view(xp, (3, 3), axis=(1, 2))[:, ::2, ::2]
    want = np.rint(win.max(axis=(-1, -2)) / d) + z
    assert np.array_equal(y, want.astype(np.uint8))


def test_global_avgpool_against_rational():
    g = np.random.default_rng(16)
    x = g.integers(0, 256, size=(3, 7, 7, 8), dtype=np.uint8)
    dx, dy, zx, zy = 0.02, 0.015, 4, 9
    M = float(np.float32(dx)) / (49 * float(np.float32(dy)))
    m, r = oracle.quantize_multiplier(M)
    y = oracle.global_avgpool_u8(x, zx, m, r, zy, c=5)
    s = x.astype(np.int64).sum(axis=(1, 2)) - 49 * zx
    for b in range(3):
        for ch in range(5):
            v = Fraction(int(s[b, ch]) * m, 2 ** r) + Fraction(1, 2)
            assert y[b, 0, 0, ch] == min(max(zy + v.numerator // v.denominator, 0), 255)
            assert abs(y[b, 0, 0, ch] - min(max(zy + s[b, ch] * M, 0), 255)) <= 0.5 + 1e-3


def test_planted_mistakes_would_be_caught():
    # The float64 pin distinguishes the defining form from common slips: dropping the
    # constant term, or counting padded taps in it.
    g = np.random.default_rng(17)
    x, wq, _ = rand_case(g, 1, 5, 5, 3, 2, 3, signed_w=False)
    z_x, z_w = 50, np.array([60, 61], np.int32)
    good = oracle.conv2d_acc(x, z_x, wq, z_w, None, 1, 1)
    xi = x.astype(np.int64)
    xpad0 = np.pad(xi, ((0, 0), (1, 1), (1, 1), (0, 0)))
    win = sliding_window_view(xpad0, (3, 3), axis=(1, 2))
    raw = np.einsum("bhwcij,oijc->bhwo", win, wq.astype(np.int64))
    sum_x = win.sum(axis=(3, 4, 5))[..., None]
    sum_w = wq.astype(np.int64).sum(axis=(1, 2, 3))
    wrong_const = raw - z_w * sum_x - z_x * sum_w + 27 * z_x * z_w      # counts padded taps
    assert not np.array_equal(good, wrong_const)
    assert np.array_equal(good[:, 1:-1, 1:-1], wrong_const[:, 1:-1, 1:-1])  # interior agrees
