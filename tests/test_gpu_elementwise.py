"""GPU parity: calibrate / quantize / dequantize / BN fold / bias / glue ops against the oracle.
Integer outputs bit-exact; floats within 1e-6 relative (in practice identical bits)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq, pitched  # noqa: F401

pytestmark = pytest.mark.gpu


def same_params(a, b):
    assert np.array_equal(a["zero_point"], b["zero_point"])
    for f in ("scale", "min_nudged", "max_nudged"):
        assert np.allclose(a[f], b[f], rtol=1e-6, atol=0), f
        assert np.array_equal(a[f], b[f]), f


@pytest.mark.parametrize("n", [1, 5, 16, 4099, 16384, 1 << 20, (1 << 22) + 3])
def test_calibrate_per_layer(hq, n):
    x = synth.normal_f32((n,), 5, n % 97, std=2.5, mean=0.7)
    same_params(hq.calibrate_minmax(dev(x)), oracle.calibrate_minmax(x))
    xp = np.abs(x) + np.float32(2.1)                       # one-sided: range is relaxed to 0
    q = hq.calibrate_minmax(dev(xp))
    same_params(q, oracle.calibrate_minmax(xp))
    assert q["zero_point"][0] == 0


def test_calibrate_misaligned_view_and_errors(hq):
    x = synth.normal_f32((10007,), 6, 1)
    base = dev(x)
    for off in (1, 2, 3):
        same_params(hq.calibrate_minmax(base[off:]), oracle.calibrate_minmax(x[off:]))
    bad = x.copy()
    bad[777] = np.nan
    with pytest.raises(qtz.QtzError) as e:
        hq.calibrate_minmax(dev(bad))
    assert e.value.code == -5
    bad[777] = -np.inf
    with pytest.raises(qtz.QtzError):
        hq.calibrate_minmax(dev(bad))
    z = np.zeros(100, np.float32)
    same_params(hq.calibrate_minmax(dev(z)), oracle.calibrate_minmax(z))


@pytest.mark.parametrize("bits", [8, 4])
def test_calibrate_per_channel_symmetric(hq, bits):
    w = synth.single_conv(seed=3, c=24, n=40)["w"]          # OHWI
    w[7] = 0
    same_params(hq.calibrate_minmax(dev(w), axis=0, bits=bits, symmetric=True),
                oracle.calibrate_minmax(w, 0, bits, True))
    wd = synth.normal_f32((3, 3, 50), 3, 9)                 # depthwise layout, channel last
    same_params(hq.calibrate_minmax(dev(wd), axis=2, bits=bits, symmetric=True),
                oracle.calibrate_minmax(wd, 2, bits, True))
    same_params(hq.calibrate_minmax(dev(w), axis=0, bits=bits, symmetric=False),
                oracle.calibrate_minmax(w, 0, bits, False))


@pytest.mark.parametrize("n", [3, 16, 1000, 65536 + 5, (1 << 21) + 17])
def test_quantize_dequantize_u8_per_layer(hq, n):
    x = synth.uniform_f32((n,), 8, 1, -1.5, 6.5)
    x[:: 97] = 0.0
    p = oracle.calibrate_minmax(x)
    want = oracle.quantize(x, p, None, 0, 255)
    got = hq.quantize_tensor(dev(x), p)
    assert np.array_equal(host(got).astype(np.int32), want)
    back = hq.dequantize(got, p)
    assert np.array_equal(host(back), oracle.dequantize(want, p, None))
    # values beyond the range saturate, NaN takes the lowest code, ties go to even
    edge = np.array([1e30, -1e30, np.inf, -np.inf, np.nan] + [(k + 0.5) * float(p["scale"][0]) for k in range(40)],
                    np.float32)
    assert np.array_equal(host(hq.quantize_tensor(dev(edge), p)).astype(np.int32),
                          oracle.quantize(edge, p, None, 0, 255))


def test_quantize_misaligned_uses_same_rule(hq):
    x = synth.uniform_f32((4099,), 8, 2, -3, 3)
    p = oracle.calibrate_minmax(x)
    got = hq.quantize_tensor(dev(x)[1:], p)
    assert np.array_equal(host(got).astype(np.int32), oracle.quantize(x[1:], p, None, 0, 255))


@pytest.mark.parametrize("restrict", [True, False])
def test_quantize_weights_s8_per_channel(hq, restrict):
    w = synth.single_conv(seed=4, c=16, n=32)["w"]
    p = oracle.calibrate_minmax(w, 0, 8, True)
    lo, hi = oracle.code_range(8, 1, int(restrict))
    want = oracle.quantize(w, p, 0, lo, hi)
    got = hq.quantize_tensor(dev(w), p, axis=0, out_dtype=qtz.S8, restrict_range=restrict)
    assert np.array_equal(host(got).astype(np.int32), want)
    assert np.array_equal(host(hq.dequantize(got, p, axis=0)), oracle.dequantize(want, p, 0))
    # depthwise layout: per-channel on the last axis
    wd = synth.normal_f32((3, 3, 40), 4, 7)
    pd = oracle.calibrate_minmax(wd, 2, 8, True)
    gd = hq.quantize_tensor(dev(wd), pd, axis=2, out_dtype=qtz.S8, restrict_range=restrict)
    assert np.array_equal(host(gd).astype(np.int32), oracle.quantize(wd, pd, 2, lo, hi))


@pytest.mark.parametrize("k", [144, 27, 9])
def test_quantize_s4_packed(hq, k):
    w = synth.normal_f32((12, k), 4, k)
    p = oracle.calibrate_minmax(w, 0, 4, True)
    codes = oracle.quantize(w, p, 0, -8, 7)
    want = oracle.pack_s4(codes)
    got = hq.quantize_tensor(dev(w), p, axis=0, out_dtype=qtz.S4_PACKED)
    assert np.array_equal(host(got).reshape(want.shape), want)
    back = hq.dequantize(got, p, axis=0, in_dtype=qtz.S4_PACKED, shape=w.shape)
    assert np.array_equal(host(back), oracle.dequantize(codes, p, 0))
    # raw packed codes containing -8 dequantize correctly as well
    raw = synth.rng(4, 99).integers(-8, 8, size=(12, k)).astype(np.int32)
    raw[0, 0] = -8
    back = hq.dequantize(dev(oracle.pack_s4(raw)), p, axis=0, in_dtype=qtz.S4_PACKED, shape=raw.shape)
    assert np.array_equal(host(back), oracle.dequantize(raw, p, 0))


def test_s4_packed_along_channels_when_inner_is_one(hq):
    wd = synth.normal_f32((9, 37), 4, 55)                     # [taps][c], per-channel on the last axis
    p = oracle.calibrate_minmax(wd, 1, 4, True)
    codes = oracle.quantize(wd, p, 1, -8, 7)
    got = hq.quantize_tensor(dev(wd), p, axis=1, out_dtype=qtz.S4_PACKED)
    assert np.array_equal(host(got).reshape(9, 19), oracle.pack_s4(codes))


def test_dequantize_int32_accumulators(hq):
    acc = synth.rng(9, 1).integers(-2 ** 31, 2 ** 31, size=(300, 24)).astype(np.int32)
    p = np.zeros(24, qtz.QPARAMS)
    p["scale"] = synth.uniform_f32((24,), 9, 2, 1e-5, 1e-2)
    got = hq.dequantize(dev(acc), p, axis=1)
    assert np.array_equal(host(got), oracle.dequantize(acc, p, 1))


def test_fold_batchnorm_and_bias(hq):
    n, k = 40, 3 * 3 * 24
    w = synth.normal_f32((n, 3, 3, 24), 10, 1)
    bn = synth.batchnorm_params(n, 10, 2)
    cb = synth.normal_f32((n,), 10, 3, std=0.2)
    for bias in (cb, None):
        w_inf, b_inf = hq.fold_batchnorm(dev(w), None if bias is None else dev(bias), dev(bn["gamma"]),
                                         dev(bn["beta"]), dev(bn["mean"]), dev(bn["var"]), 1e-3)
        ow, ob = oracle.fold_batchnorm(w, bias, bn["gamma"], bn["beta"], bn["mean"], bn["var"], 1e-3)
        assert np.allclose(host(w_inf), ow, rtol=1e-6, atol=0) and np.array_equal(host(w_inf), ow)
        assert np.allclose(host(b_inf), ob, rtol=1e-6, atol=0) and np.array_equal(host(b_inf), ob)
    wp = oracle.calibrate_minmax(ow, 0, 8, True)
    got = hq.quantize_bias(dev(ob), 0.0235, wp)
    assert np.array_equal(host(got), oracle.quantize_bias(ob, 0.0235, wp["scale"]))
    got = hq.quantize_bias(dev(ob), 0.0235, wp[:1], per_layer=True)
    assert np.array_equal(host(got), oracle.quantize_bias(ob, 0.0235, np.repeat(wp["scale"][:1], n)))


@pytest.mark.parametrize("c,pixels", [(16, 1000), (24, 333), (64, 4097)])
def test_add_u8(hq, c, pixels):
    a = pitched(synth.uniform_u8((pixels, c), 11, 1))
    b = pitched(synth.uniform_u8((pixels, c), 11, 2))
    for sa, sb, sy, za, zb, zy, relu in [(0.02, 0.031, 0.04, 3, 128, 0, True), (0.1, 0.1, 0.1, 0, 0, 0, False),
                                         (0.003, 0.05, 0.03, 255, 17, 99, False)]:
        ma, mb, r = oracle.add_params(sa, sb, sy)
        lo, hi = oracle.activation_range(1 if relu else 0, sy, zy)
        want = oracle.add_u8(a, za, ma, b, zb, mb, r, zy, lo, hi, c=c)
        got = host(hq.add_u8(dev(a), za, ma, dev(b), zb, mb, r, zy, lo, hi, c))
        assert np.array_equal(got[:, :c], want[:, :c])
    # every shift range of the kernel: 16..38 (split multipliers), above 38, 10..15 and below 10
    for ma, mb, r in [(2147483647, 1518500250, 38), (1 << 30, 3 << 28, 16), (1 << 30, 3 << 28, 40), (1200, 700, 12), (37, 21, 5),
                      (65535, 65536, 31), (0, 2147418113, 33), (1 << 30, 3 << 28, 53), (2147483647, 1 << 29, 45), (1 << 30, 1 << 30, 39)]:
        want = oracle.add_u8(a, 200, ma, b, 13, mb, r, 77, 5, 250, c=c)
        got = host(hq.add_u8(dev(a), 200, ma, dev(b), 13, mb, r, 77, 5, 250, c))
        assert np.array_equal(got[:, :c], want[:, :c])


def test_maxpool_and_global_avgpool(hq):
    x = pitched(synth.uniform_u8((3, 13, 11, 24), 12, 1))
    want = oracle.maxpool_u8(x, 3, 2, 1, c=24)
    got = host(hq.maxpool_u8(dev(x), 24, 3, 2, 1))
    assert got.shape == want.shape and np.array_equal(got[..., :24], want[..., :24])
    for shape, k, st, pad in [((2, 112, 112, 64), 3, 2, 1), ((1, 9, 12, 16), 3, 2, 0), ((2, 8, 7, 48), 3, 2, 2), ((1, 10, 10, 16), 2, 2, 0),
                              ((1, 11, 9, 32), 3, 1, 1), ((2, 12, 13, 16), 5, 2, 2), ((1, 6, 6, 16), 1, 1, 0)]:
        xx = pitched(synth.uniform_u8(shape, 12, shape[1]))
        got = host(hq.maxpool_u8(dev(xx), shape[3], k, st, pad))
        assert np.array_equal(got, oracle.maxpool_u8(xx, k, st, pad, c=shape[3]))
    x7 = pitched(synth.uniform_u8((5, 7, 7, 40), 12, 2))
    m, r = oracle.quantize_multiplier(0.02 / (49 * 0.015))
    want = oracle.global_avgpool_u8(x7, 4, m, r, 9, c=40)
    got = host(hq.global_avgpool_u8(dev(x7), 4, 9, m, r, 40))
    assert np.array_equal(got[..., :40], want[..., :40])


def test_argument_errors(hq):
    x = dev(np.zeros(64, np.float32))
    lib, h = hq.lib, hq.h
    p = np.zeros(1, qtz.QPARAMS)
    p["scale"] = 1.0
    out = torch.empty(64, dtype=torch.uint8, device="cuda")
    pp = p.ctypes.data
    assert lib.qtz_calibrate_minmax(h, None, 1, 1, 64, 8, 0, pp, None) == -1
    assert lib.qtz_calibrate_minmax(h, x.data_ptr(), 1, 1, 0, 8, 0, pp, None) == -1
    assert lib.qtz_calibrate_minmax(h, x.data_ptr(), 1, 1, 64, 17, 0, pp, None) == -1     # bits in [2,16]
    assert lib.qtz_quantize_tensor(h, x.data_ptr(), 1, 1, 64, pp, 7, 0, out.data_ptr(), None) == -1
    assert lib.qtz_quantize_tensor(h, x.data_ptr() + 2, 1, 1, 32, pp, 0, 0, out.data_ptr(), None) == -2
    p["scale"] = 0.0
    assert lib.qtz_quantize_tensor(h, x.data_ptr(), 1, 1, 64, pp, 0, 0, out.data_ptr(), None) == -1


def test_minmax_raw_range(hq):
    x = synth.normal_f32((3, 50, 7), 13, 1)
    lo, hi = hq.minmax(dev(x))
    olo, ohi = oracle.minmax(x)
    assert np.array_equal(lo, olo) and np.array_equal(hi, ohi)
    lo, hi = hq.minmax(dev(x), axis=1)
    olo, ohi = oracle.minmax(x, 1)
    assert np.array_equal(lo, olo) and np.array_equal(hi, ohi)
