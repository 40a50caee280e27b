"""Pins for the oracle's quantizer functions (Section 2.1-2.2, 2.5, 3.2.2 of the paper).

Expected values here never come from the function under test: they are the paper's
worked example, closed forms retyped in float64 / exact rationals, or invariants.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_worked_example_range_relaxation():
    # Section 2.1: (2.1, 3.5) is relaxed to (0, 3.5).
    rows = [l.split() for l in open(os.path.join(GOLDEN, "affine_worked_example.txt"))
            if l.strip() and not l.startswith("#")]
    for lo, hi, bits, rlo, rhi, z, num, den in rows:
        q = oracle.affine_params(float(lo), float(hi), int(bits))
        assert q["zero_point"] == int(z)
        assert q["scale"] == np.float32(float(num) / float(den))
        assert q["min_nudged"] == np.float32(float(rlo))
        assert abs(float(q["max_nudged"]) - float(rhi)) <= 1e-6 * float(rhi)
    # the same example through the tensor entry point
    x = np.array([2.1, 3.5, 2.7], np.float32)
    q = oracle.calibrate_minmax(x)[0]
    assert q["zero_point"] == 0 and q["scale"] == np.float32(np.float32(3.5) / 255.0)


def test_negative_one_sided_range_is_relaxed_too():
    q = oracle.affine_params(-3.5, -2.1, 8)
    assert q["zero_point"] == 255
    assert q["scale"] == np.float32(3.5 / 255.0)
    assert q["max_nudged"] == 0.0


@pytest.mark.parametrize("bits", [4, 8, 16])
def test_affine_param_invariants(bits):
    g = np.random.default_rng(7)
    L = 2 ** bits - 1
    for _ in range(2000):
        lo = float(np.float32(g.normal() * 10 ** g.uniform(-3, 3)))
        hi = float(np.float32(lo + abs(g.normal()) * 10 ** g.uniform(-3, 3)))
        q = oracle.affine_params(lo, hi, bits)
        z, d = int(q["zero_point"]), float(q["scale"])
        rlo, rhi = min(lo, 0.0), max(hi, 0.0)
        assert 0 <= z <= L
        # closed form: scale = (max - min) / (2^b - 1) on the relaxed range
        assert d == np.float32((rhi - rlo) / L)
        # z = round(-min / scale), within the code range
        assert abs(z - (-rlo / d)) <= 0.5 + 1e-6 * L
        # nudged range contains zero and is one grid step away from the real one at most
        assert q["min_nudged"] <= 0.0 <= q["max_nudged"]
        assert abs(float(q["min_nudged"]) - rlo) <= d / 2 * (1 + 1e-5) + 1e-30
        assert abs(float(q["max_nudged"]) - rhi) <= d / 2 * (1 + 1e-5) + 1e-5 * abs(rhi)
        # real zero is exactly representable: Q(0) = z and DQ(z) = 0.0
        qmin, qmax = oracle.code_range(bits, 0, 0)
        assert oracle.quantize(np.zeros(1, np.float32), q, None, qmin, qmax)[0] == z
        assert oracle.dequantize(np.array([z], np.int32), q, None)[0] == 0.0


def test_symmetric_range_gives_mid_zero_point():
    for a in [0.5, 1.0, 3.3, 117.0]:
        q = oracle.affine_params(-a, a, 8)
        assert int(q["zero_point"]) in (127, 128)


def test_degenerate_and_nonfinite():
    q = oracle.affine_params(0.0, 0.0, 8)
    assert q["scale"] == 1.0 and q["zero_point"] == 0
    q = oracle.symmetric_params(0.0, 0.0, 8)
    assert q["scale"] == 1.0 and q["zero_point"] == 0
    with pytest.raises(oracle.OracleError):
        oracle.calibrate_minmax(np.array([1.0, np.nan], np.float32))
    with pytest.raises(oracle.OracleError):
        oracle.calibrate_minmax(np.array([1.0, np.inf], np.float32))


def test_code_ranges_follow_equations():
    # Eq. 2 / Eq. 9: unsigned 0..N-1; Eq. 8: signed -N/2..N/2-1;
    # Eq. 10-11: restricted -(N/2-1)..N/2-1 and 0..N-2.
    assert oracle.code_range(8, 0, 0) == (0, 255)
    assert oracle.code_range(8, 1, 0) == (-128, 127)
    assert oracle.code_range(8, 1, 1) == (-127, 127)
    assert oracle.code_range(8, 0, 1) == (0, 254)
    assert oracle.code_range(4, 1, 0) == (-8, 7)
    assert oracle.code_range(4, 0, 0) == (0, 15)
    # the 16-bit precision of Section 7
    assert oracle.code_range(16, 0, 0) == (0, 65535)
    assert oracle.code_range(16, 1, 0) == (-32768, 32767)
    assert oracle.code_range(16, 1, 1) == (-32767, 32767)
    assert oracle.code_range(16, 0, 1) == (0, 65534)
    for bad in (1, 17):
        with pytest.raises(oracle.OracleError):
            oracle.code_range(bad, 0, 0)


def test_symmetric_params_closed_form():
    g = np.random.default_rng(3)
    w = g.normal(size=(6, 3, 3, 5)).astype(np.float32)
    w[2] = 0
    q = oracle.calibrate_minmax(w, axis=0, bits=8, symmetric=True)
    q4 = oracle.calibrate_minmax(w, axis=0, bits=4, symmetric=True)
    for n in range(6):
        a = float(np.abs(w[n]).max())
        assert q["zero_point"][n] == 0 and q4["zero_point"][n] == 0
        assert q["scale"][n] == (np.float32(a / 127.0) if a > 0 else 1.0)
        assert q4["scale"][n] == (np.float32(a / 7.0) if a > 0 else 1.0)
    # per-axis view in the middle of the tensor: channel-last (depthwise) layout
    wd = g.normal(size=(3, 3, 7)).astype(np.float32)
    qd = oracle.calibrate_minmax(wd, axis=2, bits=8, symmetric=True)
    for c in range(7):
        assert qd["scale"][c] == np.float32(float(np.abs(wd[:, :, c]).max()) / 127.0)


@pytest.mark.parametrize("bits,signed", [(8, 0), (8, 1), (4, 1), (4, 0), (16, 0), (16, 1)])
def test_quantize_against_float64_rounding(bits, signed):
    g = np.random.default_rng(11)
    x = (g.normal(size=20000) * 2.0).astype(np.float32)
    if signed:
        q = oracle.calibrate_minmax(x, bits=bits, symmetric=True)[0]
    else:
        q = oracle.calibrate_minmax(x, bits=bits)[0]
    qmin, qmax = oracle.code_range(bits, signed, 0)
    got = oracle.quantize(x, q, None, qmin, qmax)
    d, z = float(q["scale"]), int(q["zero_point"])
    t = x.astype(np.float64) / d                    # exact quotient to 2^-53
    frac = np.abs(t - np.floor(t) - 0.5)
    # away from ties the rounding rule is moot (the fp32 quotient is off by up to 2^-24 of its size: 2^-8 at 16 bits)
    safe = frac > (1e-4 if bits <= 8 else 5e-3)
    want = np.clip(np.floor(t + 0.5) + z, qmin, qmax).astype(np.int64)
    assert safe.sum() > 19000
    assert np.array_equal(got[safe], want[safe])
    assert np.all(np.abs(got[~safe] - want[~safe]) <= 1)
    assert got.min() >= qmin and got.max() <= qmax


def test_quantize_ties_round_to_even_and_saturate():
    q = np.zeros(1, oracle.QPARAMS)
    q["scale"], q["zero_point"] = 1.0, 10
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 1e30, -1e30, np.inf, -np.inf, 244.5, 245.5],
                 np.float32)
    got = oracle.quantize(x, q, None, 0, 255)
    assert got.tolist() == [10, 12, 12, 10, 8, 255, 0, 255, 0, 254, 255]
    # NaN goes to the lowest code
    assert oracle.quantize(np.array([np.nan], np.float32), q, None, 0, 255)[0] == 0


@pytest.mark.parametrize("bits", [4, 8, 16])
def test_quantize_dequantize_idempotent_and_error_bound(bits):
    g = np.random.default_rng(5)
    L = 2 ** bits - 1
    codes = np.arange(L + 1, dtype=np.int32)
    for _ in range(300 if bits <= 8 else 40):
        lo = -abs(g.normal()) * 10 ** g.uniform(-2, 2)
        hi = abs(g.normal()) * 10 ** g.uniform(-2, 2)
        q = oracle.affine_params(lo, hi, bits)
        x = oracle.dequantize(codes, q, None)
        assert np.array_equal(oracle.quantize(x, q, None, 0, L), codes)   # Q(DQ(q)) == q
        # |DQ(Q(x)) - x| <= scale/2 inside the nudged range, saturation outside
        xs = g.uniform(float(q["min_nudged"]), float(q["max_nudged"]), 500).astype(np.float32)
        back = oracle.dequantize(oracle.quantize(xs, q, None, 0, L), q, None)
        d = float(q["scale"])
        # (beyond the half step: the fp32 quotient and the fp32 product are each off by up to 2^-24 of their size,
        #  together L 2^-23 steps -- 6e-5 of a half step at 8 bits, 1.6e-2 at 16)
        assert np.all(np.abs(back.astype(np.float64) - xs) <= d / 2 * (1 + max(1e-4, 1.01 * L * 2.0 ** -22)))
        out = np.array([float(q["max_nudged"]) + 3 * d, float(q["min_nudged"]) - 3 * d],
                       np.float32)
        assert oracle.quantize(out, q, None, 0, L).tolist() == [L, 0]


def test_restricted_range_never_emits_minus_128():
    g = np.random.default_rng(9)
    w = g.normal(size=(4, 50)).astype(np.float32)
    q = oracle.calibrate_minmax(w, axis=0, symmetric=True)
    codes = oracle.quantize(w, q, 0, *oracle.code_range(8, 1, 1))
    assert codes.min() >= -127 and codes.max() <= 127
    # the extreme element of every row lands exactly on +-127
    assert np.array_equal(np.abs(codes).max(axis=1), np.full(4, 127))


def test_per_channel_codes_do_not_depend_on_power_of_two_gain():
    # Section 3.1.2: per-channel quantization makes accuracy independent of the
    # batch-norm scaling of a channel; for a power-of-two gain the codes are identical.
    g = np.random.default_rng(21)
    w = g.normal(size=(5, 3, 3, 4)).astype(np.float32)
    w2 = w.copy()
    w2[1] *= 8.0
    w2[3] *= 0.25
    r = oracle.code_range(8, 1, 1)
    c1 = oracle.quantize(w, oracle.calibrate_minmax(w, 0, 8, True), 0, *r)
    c2 = oracle.quantize(w2, oracle.calibrate_minmax(w2, 0, 8, True), 0, *r)
    assert np.array_equal(c1, c2)


def test_int4_pack_round_trip_all_bytes():
    allbytes = np.arange(256, dtype=np.uint8).reshape(16, 16)
    codes = oracle.unpack_s4(allbytes, 32)
    assert codes.min() == -8 and codes.max() == 7
    # nibble order: low nibble is the even element, two's complement
    b = 0xA3
    c = oracle.unpack_s4(np.array([[b]], np.uint8), 2)[0]
    assert c.tolist() == [3, 0xA - 16]
    assert np.array_equal(oracle.pack_s4(codes), allbytes)
    odd = np.array([[1, -2, 7]], np.int32)
    p = oracle.pack_s4(odd)
    assert p.shape == (1, 2) and np.array_equal(oracle.unpack_s4(p, 3), odd)


def test_dequantize_int32_accumulators_scale_only():
    acc = np.array([[3, -70000], [123456789, -1]], np.int32)
    q = np.zeros(2, oracle.QPARAMS)
    q["scale"] = [np.float32(0.25), np.float32(1e-3)]
    got = oracle.dequantize(acc, q, 1)
    want = acc.astype(np.float32) * q["scale"][None, :]
    assert np.array_equal(got, want)


def test_sqnr_per_channel_beats_per_layer():
    # Appendix A: SQNR = 10 log10(sum W^2 / sum (W - SimQuant(W))^2); with a wide spread
    # of per-channel gains, per-channel quantization has the higher SQNR.
    from paper_1806_08342_b200 import synth
    w = synth.single_conv(seed=1)["w"]
    r = oracle.code_range(8, 1, 1)
    qc = oracle.calibrate_minmax(w, 0, 8, True)
    wc = oracle.dequantize(oracle.quantize(w, qc, 0, *r), qc, 0)
    ql = oracle.calibrate_minmax(w, None, 8, True)
    wl = oracle.dequantize(oracle.quantize(w, ql, None, *r), ql, None)

    def sqnr(a, b):
        a = a.astype(np.float64).reshape(a.shape[0], -1)
        b = b.astype(np.float64).reshape(a.shape[0], -1)
        return 10 * np.log10((a ** 2).sum(1) / np.maximum(((a - b) ** 2).sum(1), 1e-300))
    sc, sl = sqnr(w, wc), sqnr(w, wl)
    assert np.all(sc > 35.0)            # 8-bit uniform on a Gaussian kernel: roughly 40 dB
    assert np.median(sc) > np.median(sl) + 6.0
    assert sl.min() < 20.0              # the small-gain channels collapse per layer
