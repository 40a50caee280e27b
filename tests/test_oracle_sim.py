"""Pins for the oracle's quantizer utilities: SimQuant (Section 2.4), SQNR (Appendix A), the moving
average of activation ranges (Section 2.5) and the rescale to another quantizer (concat, Section 3.2.1).

Expected values never come from the function under test: closed forms in float64 or exact
rationals, textbook results, hand-computed numbers, invariants.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _params(lo, hi, bits=8):
    return oracle.affine_params(lo, hi, bits)


def test_simquant_closed_form_away_from_ties():
    g = np.random.default_rng(3)
    x = g.uniform(-2.0, 7.0, 20000).astype(np.float32)
    p = _params(-1.0, 6.0)
    d, z = float(p["scale"]), int(p["zero_point"])
    y = oracle.simquant(x, p, None, 0, 255)
    t = x.astype(np.float64) / d
    far = np.abs(t - np.floor(t) - 0.5) > 1e-4            # fp32 division may land on the other side of a tie
    want = d * (np.clip(np.rint(t) + z, 0, 255) - z)
    assert np.allclose(y[far], want[far], rtol=1e-6, atol=1e-7)
    assert far.sum() > 19000


def test_simquant_is_idempotent_and_bounded():
    g = np.random.default_rng(4)
    x = g.normal(0.0, 1.0, 5000).astype(np.float32)
    p = _params(float(x.min()), float(x.max()))
    d = float(p["scale"])
    y = oracle.simquant(x, p, None, 0, 255)
    assert np.array_equal(oracle.simquant(y, p, None, 0, 255), y)          # a code's real value maps to itself
    inside = (x >= p["min_nudged"]) & (x <= p["max_nudged"])
    assert np.all(np.abs(y[inside].astype(np.float64) - x[inside]) <= d / 2 * (1 + 1e-5))
    assert np.all(y[x > p["max_nudged"]] == p["max_nudged"])
    assert np.all(y[x < p["min_nudged"]] == p["min_nudged"])
    assert oracle.simquant(np.zeros(3, np.float32), p, None, 0, 255).tolist() == [0.0, 0.0, 0.0]   # real zero is exact


def test_simquant_per_channel_symmetric_weights():
    g = np.random.default_rng(5)
    w = (g.normal(0, 1, (6, 3, 3, 4)) * np.array([0.1, 1, 3, 0.5, 2, 8]).reshape(6, 1, 1, 1)).astype(np.float32)
    q = oracle.calibrate_minmax(w, axis=0, symmetric=True)
    y = oracle.simquant(w, q, 0, -127, 127)
    for n in range(6):
        d = float(q[n]["scale"])
        assert d == np.float32(np.abs(w[n]).max() / 127.0)
        codes = y[n].astype(np.float64) / d
        assert np.allclose(codes, np.rint(codes), atol=1e-3) and np.abs(codes).max() <= 127.0 + 1e-3


def test_sqnr_hand_computed():
    w = np.array([1.0, 2.0], np.float32)
    wh = np.array([1.0, 1.5], np.float32)
    assert abs(oracle.sqnr(w, wh)[0] - 10 * math.log10(5.0 / 0.25)) < 1e-12
    per = oracle.sqnr(np.array([[3.0, 4.0], [1.0, 0.0]], np.float32), np.array([[3.0, 3.0], [0.5, 0.0]], np.float32), axis=0)
    assert abs(per[0] - 10 * math.log10(25.0 / 1.0)) < 1e-12 and abs(per[1] - 10 * math.log10(1.0 / 0.25)) < 1e-12
    assert oracle.sqnr(w, w)[0] == math.inf
    # the ratio does not change when both tensors are scaled
    assert abs(oracle.sqnr(4 * w, 4 * wh)[0] - oracle.sqnr(w, wh)[0]) < 1e-12


@pytest.mark.parametrize("bits", [4, 8, 16])
def test_sqnr_of_a_uniform_signal_is_the_textbook_value(bits):
    # uniform on [0, R] quantized over exactly that range: noise power Delta^2 / 12, signal power R^2 / 3,
    # so SQNR = 20 log10(2 (2^b - 1))  (about 6.02 dB per bit)
    g = np.random.default_rng(6)
    x = g.uniform(0.0, 6.0, 1 << 20).astype(np.float32)
    x[0], x[1] = 0.0, 6.0
    p = _params(0.0, 6.0, bits)
    got = oracle.sqnr(x, oracle.simquant(x, p, None, 0, (1 << bits) - 1))[0]
    assert abs(got - 20 * math.log10(2 * ((1 << bits) - 1))) < 0.05


def test_per_channel_quantization_improves_sqnr_when_ranges_differ():
    # Appendix A: per-channel beats per-layer when the channels' dynamic ranges differ
    g = np.random.default_rng(7)
    w = (g.normal(0, 1, (8, 64)) * np.geomspace(0.05, 5.0, 8).reshape(8, 1)).astype(np.float32)
    layer = oracle.calibrate_minmax(w, symmetric=True)
    chan = oracle.calibrate_minmax(w, axis=0, symmetric=True)
    s_layer = oracle.sqnr(w, oracle.simquant(w, layer, None, -127, 127), axis=0)
    s_chan = oracle.sqnr(w, oracle.simquant(w, chan, 0, -127, 127), axis=0)
    assert np.all(s_chan[:6] > s_layer[:6] + 3.0) and np.all(s_chan >= s_layer - 1e-9)


def test_ema_closed_forms():
    lo, hi = np.zeros(2), np.zeros(2)
    init = oracle.ema_update(lo, hi, [-1.0, -2.0], [3.0, 4.0], 0.9, False)
    assert init and lo.tolist() == [-1.0, -2.0] and hi.tolist() == [3.0, 4.0]      # the first batch sets the state
    for _ in range(5):                                                              # a constant stays put
        oracle.ema_update(lo, hi, [-1.0, -2.0], [3.0, 4.0], 0.9, True)
    assert np.allclose(lo, [-1.0, -2.0], rtol=0, atol=1e-15) and np.allclose(hi, [3.0, 4.0], rtol=0, atol=1e-15)
    # step to a new constant v from s0: s_n = d^n s0 + (1 - d^n) v
    s = np.array([2.0]); t = np.array([10.0])
    for n in range(1, 30):
        oracle.ema_update(s, t, [0.0], [20.0], 0.8, True)
        assert abs(s[0] - (0.8 ** n * 2.0)) < 1e-12 and abs(t[0] - (0.8 ** n * 10.0 + (1 - 0.8 ** n) * 20.0)) < 1e-12
    # no memory: the last batch
    oracle.ema_update(s, t, [-7.0], [7.0], 0.0, True)
    assert s[0] == -7.0 and t[0] == 7.0
    with pytest.raises(oracle.OracleError):
        oracle.ema_update(s, t, [float("nan")], [1.0], 0.5, True)
    with pytest.raises(oracle.OracleError):
        oracle.ema_update(s, t, [0.0], [1.0], 1.0, True)


def test_rescale_identity_and_exact_rationals():
    g = np.random.default_rng(8)
    x = g.integers(0, 256, (5, 7, 16)).astype(np.uint8)
    m, r = oracle.quantize_multiplier(1.0)
    assert np.array_equal(oracle.rescale_u8(x, 9, m, r, 9), x)                       # the same quantizer: nothing changes
    m, r = oracle.quantize_multiplier(0.25)                                          # a power of two: an exact rounding shift
    y = oracle.rescale_u8(x, 0, m, r, 0)
    assert np.array_equal(y, (x.astype(np.int64) + 2) >> 2)
    real = 0.7315
    m, r = oracle.quantize_multiplier(real)
    y = oracle.rescale_u8(x, 100, m, r, 120, 10, 250, c=12).astype(np.int64)
    for idx in np.ndindex(5, 7, 12):
        exact = Fraction(int(x[idx]) - 100) * Fraction(m, 1 << r) + 120
        want = min(max(math.floor(exact + Fraction(1, 2)), 10), 250)
        assert y[idx] == want
    assert np.all(y[..., 12:] == 0)                                                  # the pitch padding is left alone
    # into a channel slice of a wider tensor
    cat = np.zeros((5, 7, 48), np.uint8)
    oracle.rescale_u8(x, 100, m, r, 120, 10, 250, c=12, out=cat, out_offset=16)
    assert np.array_equal(cat[..., 16:28], y[..., :12]) and not cat[..., :16].any() and not cat[..., 28:].any()
