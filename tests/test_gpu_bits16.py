"""GPU parity of the 16-bit precision (Section 7 recommends 4, 8 and 16 bits): quantizer parameters,
quantize, de-quantize and SimQuant with uint16 / int16 codes, bit-exact against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq  # noqa: F401

pytestmark = pytest.mark.gpu


def same_params(a, b):
    for f in ("scale", "zero_point", "min_nudged", "max_nudged"):
        assert np.array_equal(a[f], b[f]), f


@pytest.mark.parametrize("n", [1, 7, 8, 4099, 1 << 20, (1 << 21) + 5])
def test_u16_per_layer_round_trip(hq, n):
    x = synth.uniform_f32((n,), 8, 3, -1.5, 6.5)
    x[::97] = 0.0
    p = oracle.calibrate_minmax(x, bits=16)
    same_params(hq.calibrate_minmax(dev(x), bits=16), p)
    want = oracle.quantize(x, p, None, 0, 65535)
    got = hq.quantize_tensor(dev(x), p, out_dtype=qtz.U16)
    assert got.dtype == torch.uint16
    assert np.array_equal(host(got).astype(np.int32), want)
    back = hq.dequantize(got, p)
    assert np.array_equal(host(back).view(np.uint32), oracle.dequantize(want, p, None).view(np.uint32))
    # saturation, NaN to the lowest code, ties to even (the tie points are exact in fp32 for a power-of-two scale)
    q2 = np.zeros(1, oracle.QPARAMS)
    q2["scale"], q2["zero_point"] = 2.0 ** -10, 1000
    edge = np.array([1e30, -1e30, np.inf, -np.inf, np.nan] + [(k + 0.5) * 2.0 ** -10 for k in range(-40, 40)], np.float32)
    for restrict, top in ((False, 65535), (True, 65534)):
        assert np.array_equal(host(hq.quantize_tensor(dev(edge), q2, out_dtype=qtz.U16, restrict_range=restrict)).astype(np.int32),
                              oracle.quantize(edge, q2, None, 0, top))


def test_u16_misaligned_views(hq):
    x = synth.uniform_f32((4099,), 8, 4, -3, 3)
    p = oracle.calibrate_minmax(x, bits=16)
    for off in (1, 2, 3):
        got = hq.quantize_tensor(dev(x)[off:], p, out_dtype=qtz.U16)
        want = oracle.quantize(x[off:], p, None, 0, 65535)
        assert np.array_equal(host(got).astype(np.int32), want)
        codes = torch.from_numpy(want.astype(np.uint16)).cuda()
        base = torch.zeros(want.size + 8, dtype=torch.uint16, device="cuda")
        base[off:off + want.size] = codes                    # a 2-byte aligned, not 16-byte aligned, view
        assert np.array_equal(host(hq.dequantize(base[off:off + want.size], p)), oracle.dequantize(want, p, None))


@pytest.mark.parametrize("restrict", [True, False])
def test_s16_per_channel_weights(hq, restrict):
    w = synth.single_conv(seed=4, c=16, n=32)["w"]                  # OHWI
    p = oracle.calibrate_minmax(w, 0, 16, True)
    same_params(hq.calibrate_minmax(dev(w), axis=0, bits=16, symmetric=True), p)
    lo, hi = oracle.code_range(16, 1, int(restrict))
    want = oracle.quantize(w, p, 0, lo, hi)
    got = hq.quantize_tensor(dev(w), p, axis=0, out_dtype=qtz.S16, restrict_range=restrict)
    assert got.dtype == torch.int16
    assert np.array_equal(host(got).astype(np.int32), want)
    assert np.array_equal(host(hq.dequantize(got, p, axis=0)), oracle.dequantize(want, p, 0))
    wd = synth.normal_f32((3, 3, 40), 4, 7)                         # depthwise layout: channel last
    pd = oracle.calibrate_minmax(wd, 2, 16, True)
    gd = hq.quantize_tensor(dev(wd), pd, axis=2, out_dtype=qtz.S16, restrict_range=restrict)
    assert np.array_equal(host(gd).astype(np.int32), oracle.quantize(wd, pd, 2, lo, hi))
    # a flat symmetric tensor takes the vectorised kernels
    flat = synth.normal_f32((1 << 16,), 4, 8)
    pf = oracle.calibrate_minmax(flat, None, 16, True)
    gf = hq.quantize_tensor(dev(flat), pf, out_dtype=qtz.S16, restrict_range=restrict)
    wf = oracle.quantize(flat, pf, None, lo, hi)
    assert np.array_equal(host(gf).astype(np.int32), wf)
    assert np.array_equal(host(hq.dequantize(gf, pf)), oracle.dequantize(wf, pf, None))


def test_simquant_16_bits_and_its_sqnr(hq):
    x = synth.uniform_f32((1 << 20,), 8, 5, 0.0, 6.0)
    x[0], x[1] = 0.0, 6.0
    p = oracle.affine_params(0.0, 6.0, 16)
    got = hq.simquant(dev(x), p, code_dtype=qtz.U16)
    want = oracle.simquant(x, p, None, 0, 65535)
    assert np.array_equal(host(got).view(np.uint32), want.view(np.uint32))
    # uniform signal over exactly the quantizer's range: 20 log10(2 (2^16 - 1)) dB, 48.2 dB above the 8-bit figure
    db = float(hq.sqnr(dev(x), got)[0])
    assert abs(db - 20 * math.log10(2 * 65535)) < 0.05
    p8 = oracle.affine_params(0.0, 6.0, 8)
    db8 = float(hq.sqnr(dev(x), hq.simquant(dev(x), p8))[0])
    assert abs((db - db8) - 20 * math.log10(65535 / 255)) < 0.1
    w = synth.single_conv(seed=4, c=24, n=40)["w"]
    q = oracle.calibrate_minmax(w, 0, 16, True)
    got = host(hq.simquant(dev(w), q, axis=0, code_dtype=qtz.S16, restrict_range=True))
    assert np.array_equal(got.view(np.uint32), oracle.simquant(w, q, 0, -32767, 32767).view(np.uint32))


def test_bits_and_alignment_errors(hq):
    x = dev(synth.uniform_f32((64,), 8, 6, -1, 1))
    for bits in (1, 17):
        with pytest.raises(qtz.QtzError):
            hq.calibrate_minmax(x, bits=bits)
        with pytest.raises(qtz.QtzError):
            qtz.params_from_range(-1.0, 1.0, bits)
    p = np.atleast_1d(oracle.affine_params(-1.0, 1.0, 16))
    raw = torch.zeros(2 * 64 + 2, dtype=torch.uint8, device="cuda")
    odd = raw[1:1 + 128]                                           # odd address: not a uint16 array
    rc = hq.lib.qtz_quantize_tensor(hq.h, x.data_ptr(), 1, 1, 64, p.ctypes.data, qtz.U16, 0, odd.data_ptr(), None)
    assert rc == -2                                                # QTZ_ERR_MISALIGNED
