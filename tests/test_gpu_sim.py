"""GPU parity: SimQuant, SQNR and the rescale to another quantizer against the oracle.
SimQuant values and rescaled codes bit-exact; SQNR (fp64 sums in another order) within 1e-9 dB."""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq, pitched  # noqa: F401

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 15, 16, 4099, (1 << 20) + 5])
def test_simquant_per_layer(hq, n):
    x = synth.normal_f32((n,), 41, n % 89, std=2.0, mean=0.5)
    x[:: max(1, n // 7)] *= 3.0                                      # some values saturate
    p = oracle.affine_params(-3.0, 5.0)
    got = host(hq.simquant(dev(x), p))
    want = oracle.simquant(x, p, None, 0, 255)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    if n > 8:                                                         # a view that is not 16-byte aligned
        got = host(hq.simquant(dev(x)[1:], p))
        assert np.array_equal(got.view(np.uint32), want[1:].view(np.uint32))


def test_simquant_in_place_and_special_values(hq):
    x = np.array([0.0, -0.0, 1e-9, -1e-9, np.inf, -np.inf, np.nan, 2.5, -2.5, 100.0, -100.0] * 3, np.float32)
    p = oracle.affine_params(-2.0, 3.0)
    t = dev(x)
    hq.simquant(t, p, out=t)
    want = oracle.simquant(x, p, None, 0, 255)
    assert np.array_equal(host(t).view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("bits,dtype,lo,hi,restrict", [(8, qtz.S8, -127, 127, True), (4, qtz.S4_PACKED, -8, 7, False)])
def test_simquant_per_channel_weights(hq, bits, dtype, lo, hi, restrict):
    w = synth.single_conv(seed=4, c=24, n=40)["w"]                   # OHWI
    q = oracle.calibrate_minmax(w, 0, bits, True)
    got = host(hq.simquant(dev(w), q, axis=0, code_dtype=dtype, restrict_range=restrict))
    want = oracle.simquant(w, q, 0, lo, hi)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    wd = synth.normal_f32((3, 3, 50), 4, 9)                          # depthwise layout, channel last
    q = oracle.calibrate_minmax(wd, 2, bits, True)
    got = host(hq.simquant(dev(wd), q, axis=2, code_dtype=dtype, restrict_range=restrict))
    assert np.array_equal(got.view(np.uint32), oracle.simquant(wd, q, 2, lo, hi).view(np.uint32))


def test_sqnr_matches_oracle(hq):
    w = synth.single_conv(seed=5, c=32, n=48)["w"]
    for axis, sym in ((0, True), (None, True), (None, False)):
        q = oracle.calibrate_minmax(w, axis, 8, sym)
        lo, hi = (-127, 127) if sym else (0, 255)
        wh = oracle.simquant(w, q, axis, lo, hi)
        got = hq.sqnr(dev(w), dev(wh), axis=axis)
        want = oracle.sqnr(w, wh, axis)
        assert got.shape == want.shape
        assert np.allclose(got, want, rtol=0, atol=1e-9)
    big = synth.normal_f32(((1 << 21) + 3,), 5, 2)
    p = oracle.calibrate_minmax(big)
    bh = oracle.simquant(big, p, None, 0, 255)
    assert abs(hq.sqnr(dev(big), dev(bh))[0] - oracle.sqnr(big, bh)[0]) < 1e-9
    assert hq.sqnr(dev(big), dev(big))[0] == np.inf
    wd = synth.normal_f32((3, 3, 50), 5, 9)                          # channel-last view
    q = oracle.calibrate_minmax(wd, 2, 4, True)
    wh = oracle.simquant(wd, q, 2, -8, 7)
    assert np.allclose(hq.sqnr(dev(wd), dev(wh), axis=2), oracle.sqnr(wd, wh, 2), rtol=0, atol=1e-9)


@pytest.mark.parametrize("c,pitch", [(16, 16), (12, 16), (7, 16), (64, 64)])
def test_rescale_matches_oracle(hq, c, pitch):
    x = pitched(synth.uniform_u8((3, 9, 11, c), 61, c), pitch)
    for real, zx, zy, lo, hi in ((0.7315, 100, 120, 10, 250), (1.0, 9, 9, 0, 255), (3.3, 128, 5, 0, 255), (0.01, 0, 255, 0, 255)):
        m, r = oracle.quantize_multiplier(real)
        got = host(hq.rescale_u8(dev(x), zx, m, r, zy, lo, hi, c=c))
        want = oracle.rescale_u8(x, zx, m, r, zy, lo, hi, c=c)
        assert np.array_equal(got[..., :c], want[..., :c])


def test_concat_by_rescaling_into_channel_slices(hq):
    a = synth.uniform_u8((2, 5, 6, 32), 62, 1)
    b = synth.uniform_u8((2, 5, 6, 20), 62, 2)
    b = pitched(b, 32)
    ma, ra = oracle.quantize_multiplier(0.02 / 0.05)
    mb, rb = oracle.quantize_multiplier(0.05 / 0.05)
    cat_want = np.zeros((2, 5, 6, 64), np.uint8)
    oracle.rescale_u8(a, 3, ma, ra, 17, out=cat_want, out_offset=0)
    oracle.rescale_u8(b, 40, mb, rb, 17, c=20, out=cat_want, out_offset=32)
    cat = torch.zeros((2, 5, 6, 64), dtype=torch.uint8, device="cuda")
    hq.rescale_u8(dev(a), 3, ma, ra, 17, out=cat, out_offset=0)
    hq.rescale_u8(dev(b), 40, mb, rb, 17, c=20, out=cat, out_offset=32)
    assert np.array_equal(host(cat), cat_want)
    # an odd channel offset takes the byte path
    cat2 = torch.zeros((2, 5, 6, 64), dtype=torch.uint8, device="cuda")
    want2 = np.zeros((2, 5, 6, 64), np.uint8)
    oracle.rescale_u8(b, 40, mb, rb, 17, c=20, out=want2, out_offset=5)
    hq.rescale_u8(dev(b), 40, mb, rb, 17, c=20, out=cat2, out_offset=5)
    assert np.array_equal(host(cat2), want2)
