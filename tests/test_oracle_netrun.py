"""Pins of the network-level oracle (oracle/netrun.py and the range rules in qtz_oracle_net.c).

None of the expected values below comes from the functions under test:
  * the float network (batch norm folded in float64, no quantization anywhere) is evaluated in
    float64 by a few lines of numpy, and every dequantized tensor of the integer network must stay
    within a signal-to-noise bound of it (Appendix A's SQNR) -- a wrong tensor wiring, stride,
    padding value, bias scale, clamp or range rule collapses that ratio;
  * the quantizer of every convolution output is re-derived by hand: exact accumulators from a
    float64 convolution of the integer codes, the fp32 scale product, min/max over the calibration
    images only, the activation applied to both ends, then Delta = (max - min) / 255 and
    z = round(-min / Delta) (Section 2.1);
  * the range rules are checked against the textbook definitions of ReLU / ReLU6 applied to the ends
    of an interval, and the add rule against the property it exists for: no pair of representable
    inputs can saturate the output.
"""
import numpy as np
import pytest

import oracle
from oracle import netrun
from paper_1806_08342_b200 import synth

SEED = 5


def tiny_network():
    ops = []
    synth._conv(ops, "in", "t0", 3, 8, 3, 2, 2)                       # stem, ReLU6
    synth._conv(ops, "t0", "d1", 8, 8, 3, 1, 2, depthwise=True)       # depthwise, ReLU6
    synth._conv(ops, "d1", "p1", 8, 8, 1, 1, 0)                       # linear bottleneck
    ops.append({"op": "add", "a": "p1", "b": "t0", "dst": "r1", "act": 0})
    synth._conv(ops, "r1", "c2", 8, 16, 1, 1, 1)                      # ReLU
    synth._conv(ops, "c2", "c3", 16, 8, 3, 1, 0)
    ops.append({"op": "add", "a": "c3", "b": "r1", "dst": "r2", "act": 1})
    ops.append({"op": "maxpool", "src": "r2", "dst": "m", "k": 3, "stride": 2, "pad": 1})
    ops.append({"op": "avgpool", "src": "m", "dst": "pool"})
    ops.append({"op": "fc", "src": "pool", "dst": "logits", "cin": 8, "cout": 10})
    return ops


def act_f(v, kind):
    if kind == 0:
        return v
    v = np.maximum(v, 0.0)
    return np.minimum(v, 6.0) if kind == 2 else v


def conv_f64(x, w, stride, pad, depthwise):
    """x [B,H,W,C] float64, w OHWI (depthwise: HWC); out-of-image taps contribute real zero."""
    b, h, ww, c = x.shape
    kh, kw = (w.shape[0], w.shape[1]) if depthwise else (w.shape[1], w.shape[2])
    oh, ow = (h + 2 * pad - kh) // stride + 1, (ww + 2 * pad - kw) // stride + 1
    xp = np.zeros((b, h + 2 * pad, ww + 2 * pad, c))
    xp[:, pad:pad + h, pad:pad + ww] = x
    out = np.zeros((b, oh, ow, c if depthwise else w.shape[0]))
    for i in range(kh):
        for j in range(kw):
            patch = xp[:, i:i + (oh - 1) * stride + 1:stride, j:j + (ow - 1) * stride + 1:stride]
            out += patch * w[i, j] if depthwise else patch @ w[:, i, j, :].T
    return out


def float_weights(op, index):
    """The float layer: BN folded in float64 (gamma w / sigma, beta - gamma mu / sigma)."""
    raw = synth.layer_params(op, index, SEED)
    w = raw["w"].astype(np.float64)
    if "bn" not in raw:
        return w, raw["bias"].astype(np.float64)
    bn = {k: v.astype(np.float64) for k, v in raw["bn"].items()}
    g = bn["gamma"] / np.sqrt(bn["var"] + 1e-3)
    w = w * g if op["depthwise"] else w * g[:, None, None, None]
    return w, bn["beta"] - g * bn["mean"]


def float_forward(ops, images):
    t = {"in": images.astype(np.float64) / 255.0}
    for index, op in enumerate(ops):
        kind = op["op"]
        if kind == "conv":
            w, bias = float_weights(op, index)
            t[op["dst"]] = act_f(conv_f64(t[op["src"]], w, op["stride"], op["pad"], op["depthwise"]) + bias, op["act"])
        elif kind == "fc":
            w, bias = float_weights(op, index)
            t[op["dst"]] = (conv_f64(t[op["src"]], w, 1, 0, False) + bias).reshape(images.shape[0], -1)
        elif kind == "add":
            t[op["dst"]] = act_f(t[op["a"]] + t[op["b"]], op["act"])
        elif kind == "maxpool":
            x, k, s, p = t[op["src"]], op["k"], op["stride"], op["pad"]
            b, h, w_, c = x.shape
            oh, ow = (h + 2 * p - k) // s + 1, (w_ + 2 * p - k) // s + 1
            xp = np.full((b, h + 2 * p, w_ + 2 * p, c), -np.inf)
            xp[:, p:p + h, p:p + w_] = x
            t[op["dst"]] = np.max([xp[:, i:i + (oh - 1) * s + 1:s, j:j + (ow - 1) * s + 1:s]
                                   for i in range(k) for j in range(k)], axis=0)
        elif kind == "avgpool":
            t[op["dst"]] = t[op["src"]].mean(axis=(1, 2), keepdims=True)
    return t


def sqnr_db(ref, test):
    return 10.0 * np.log10(np.sum(ref * ref) / max(np.sum((ref - test) ** 2), 1e-300))


@pytest.fixture(scope="module")
def tiny():
    ops = tiny_network()
    images = synth.network_input(4, 16, SEED)
    return ops, images, netrun.run(ops, images, 2, SEED, 8)


def test_integer_network_tracks_the_float_network(tiny):
    ops, images, got = tiny
    want = float_forward(ops, images)
    worst = {}
    for name, ref in want.items():
        if name == "logits":
            continue
        rec = got[name]
        deq = (rec["q"].astype(np.float64) - float(rec["p"]["zero_point"])) * float(rec["p"]["scale"])
        assert deq.shape == ref.shape, name
        worst[name] = sqnr_db(ref, deq)
    # 8-bit weights and activations: every tensor of this network stays above 30 dB (measured 31.9-39.1 dB);
    # a mis-wired tensor, a dropped bias or clamp, or padding with code 0 instead of z_x falls far below
    assert min(worst.values()) > 30.0, worst
    assert worst["in"] > 140.0                                       # the image codes ARE the reals k/255


def test_logits_follow_the_float_classifier(tiny):
    ops, images, got = tiny
    want = float_forward(ops, images)["logits"]
    fc_index = len(ops) - 1
    codes, wq, _ = netrun.quantized_weights(ops[fc_index], fc_index, SEED, 8)
    scale = float(got["pool"]["p"]["scale"]) * wq["scale"].astype(np.float64)
    deq = got["logits"]["q"].astype(np.float64) * scale
    assert sqnr_db(want, deq) > 20.0
    assert got["logits"]["q"].dtype == np.int32 and got["logits"]["p"] is None


def test_conv_output_quantizers_rederived_by_hand(tiny):
    ops, images, got = tiny
    calib = 2
    for index, op in enumerate(ops):
        if op["op"] != "conv":
            continue
        x = got[op["src"]]
        codes, wq, bias = netrun.quantized_weights(op, index, SEED, 8)
        xs = np.float32(x["p"]["scale"])
        # exact accumulators of the calibration images: float64 convolution of (x_Q - z_x) and w_Q, plus the bias
        xr = x["q"][:calib].astype(np.float64) - float(x["p"]["zero_point"])
        acc = conv_f64(xr, codes.astype(np.float64), op["stride"], op["pad"], op["depthwise"])
        bias_q = np.rint(bias.astype(np.float64) / (np.float64(xs) * wq["scale"].astype(np.float64)))
        acc = acc + bias_q
        assert np.all(acc == np.rint(acc)) and np.abs(acc).max() < 2 ** 31
        real = acc.astype(np.float32) * (xs * wq["scale"])            # one fp32 product, one fp32 multiply
        lo, hi = act_f(np.float64(real.min()), op["act"]), act_f(np.float64(real.max()), op["act"])
        lo, hi = min(lo, 0.0), max(hi, 0.0)                            # Section 2.1: the range must hold 0
        delta = np.float32((hi - lo) / 255.0)
        z = int(np.clip(np.rint(-lo / np.float64(delta)), 0, 255))
        p = got[op["dst"]]["p"]
        assert np.float32(p["scale"]) == delta and int(p["zero_point"]) == z, (op["dst"], p, delta, z)
        assert np.float32(p["min_nudged"]) == np.float32(-z) * delta
        assert np.float32(p["max_nudged"]) == np.float32(255 - z) * delta


def test_range_after_activation_is_the_interval_image():
    rng = synth.rng(77, 0)
    cases = [(-3.0, 9.0), (-3.0, 4.0), (1.0, 9.0), (7.0, 9.0), (-5.0, -1.0), (0.0, 0.0), (-2.5, 6.0), (6.0, 6.5)]
    cases += [tuple(sorted(rng.uniform(-10, 10, 2))) for _ in range(200)]
    for lo, hi in cases:
        lo, hi = float(np.float32(lo)), float(np.float32(hi))
        for kind in (0, 1, 2):
            got = oracle.range_after_activation(lo, hi, kind)
            xs = np.linspace(lo, hi, 257)
            img = act_f(xs, kind)
            assert got == (float(img.min()), float(img.max())), (lo, hi, kind, got)   # tight: both ends attained
    with pytest.raises(oracle.OracleError):
        oracle.range_after_activation(2.0, 1.0, 0)
    with pytest.raises(oracle.OracleError):
        oracle.range_after_activation(float("nan"), 1.0, 1)


def test_relu6_clamp_codes_sit_on_real_zero_and_six():
    for lo, hi in [(-1.3, 7.7), (-0.2, 5.1), (0.0, 6.0), (-4.0, 6.0)]:
        p = oracle.affine_params(*oracle.range_after_activation(lo, hi, 2), 8)
        amin, amax = oracle.activation_range(2, p["scale"], int(p["zero_point"]))
        assert (amin - int(p["zero_point"])) * float(p["scale"]) == 0.0
        top = (amax - int(p["zero_point"])) * float(p["scale"])
        assert abs(top - min(6.0, max(hi, 0.0))) <= 0.5 * float(p["scale"]) * 1.0001


def test_add_range_cannot_saturate():
    rng = synth.rng(78, 0)
    for _ in range(60):
        pa = oracle.affine_params(*sorted(np.float32(rng.uniform(-8, 8, 2))), 8)
        pb = oracle.affine_params(*sorted(np.float32(rng.uniform(-3, 12, 2))), 8)
        lo, hi = oracle.add_output_range(pa, pb, 0)
        # interval arithmetic on what the inputs can represent, to fp32 rounding
        assert lo == float(np.float32(pa["min_nudged"]) + np.float32(pb["min_nudged"]))
        assert hi == float(np.float32(pa["max_nudged"]) + np.float32(pb["max_nudged"]))
        py = oracle.affine_params(lo, hi, 8)
        ma, mb, r = oracle.add_params(pa["scale"], pb["scale"], py["scale"])
        qa = np.array([[0, 0, 255, 255, int(pa["zero_point"]), 17]], np.uint8)
        qb = np.array([[0, 255, 0, 255, int(pb["zero_point"]), 200]], np.uint8)
        y = oracle.add_u8(qa, int(pa["zero_point"]), ma, qb, int(pb["zero_point"]), mb, r, int(py["zero_point"]), 0, 255)
        real = ((qa.astype(np.float64) - int(pa["zero_point"])) * float(pa["scale"]) +
                (qb.astype(np.float64) - int(pb["zero_point"])) * float(pb["scale"]))
        back = (y.astype(np.float64) - int(py["zero_point"])) * float(py["scale"])
        # never clipped: every extreme pair lands within one output step of its real sum
        assert np.all(np.abs(back - real) <= 1.01 * float(py["scale"])), (real, back)
        # with ReLU the range is the same interval pushed through max(., 0)
        assert oracle.add_output_range(pa, pb, 1) == (max(lo, 0.0), max(hi, 0.0))


def test_pooling_keeps_the_quantizer_and_means_of_constants(tiny):
    ops, images, got = tiny
    assert got["m"]["p"].tobytes() == got["r2"]["p"].tobytes()
    assert got["pool"]["p"].tobytes() == got["m"]["p"].tobytes()
    p = got["m"]["p"]
    const = {"src": QT(np.full((2, 5, 5, 8), 77, np.uint8), p)}
    out = netrun.op_avgpool({"op": "avgpool", "src": "src", "dst": "o"}, 0, const, {})
    assert np.all(out.q == 77)                                        # the mean of a constant is the constant
    ramp = np.arange(2 * 4 * 4 * 8, dtype=np.int64).reshape(2, 4, 4, 8) % 251
    out = netrun.op_avgpool({"op": "avgpool", "src": "src", "dst": "o"}, 0,
                            {"src": QT(ramp.astype(np.uint8), p)}, {})
    z = int(p["zero_point"])
    mean = np.floor((ramp - z).reshape(2, 16, 8).sum(axis=1) / 16.0 + 0.5) + z      # ties toward +inf
    assert np.array_equal(out.q.reshape(2, 8), np.clip(mean, 0, 255).astype(np.uint8))


def QT(q, p):
    return netrun.QTensor(q, p)


def test_streaming_mode_and_visitor_agree_with_the_kept_run(tiny):
    ops, images, got = tiny
    seen = {}
    out = netrun.run(ops, images, 2, SEED, 8, visit=lambda name, t: seen.__setitem__(name, t.q.copy()), keep=False)
    assert set(seen) == set(got)
    for name in got:
        assert np.array_equal(seen[name], got[name]["q"]), name
    assert np.array_equal(out["logits"]["q"], got["logits"]["q"])
    assert "t0" not in out                                             # dropped once nothing reads it


def test_four_bit_weights_go_through_the_packed_form():
    ops = tiny_network()
    images = synth.network_input(2, 16, SEED)
    got = netrun.run(ops, images, 2, SEED, 4)
    codes, wq, _ = netrun.quantized_weights(ops[0], 0, SEED, 4)
    assert codes.min() >= -8 and codes.max() <= 7 and len(np.unique(codes)) > 8
    want = float_forward(ops, images)
    deq = (got["t0"]["q"].astype(np.float64) - float(got["t0"]["p"]["zero_point"])) * float(got["t0"]["p"]["scale"])
    assert 8.0 < sqnr_db(want["t0"], deq) < 40.0                       # 4-bit weights: coarser than 8-bit, still a signal


def test_planted_mistakes_in_the_network_oracle_would_be_caught(monkeypatch):
    """Each plausible slip, planted in the oracle on the CPU, breaks one of the pins above."""
    ops = tiny_network()
    images = synth.network_input(4, 16, SEED)
    want = float_forward(ops, images)

    def worst_sqnr(got):
        vals = []
        for name, ref in want.items():
            if name in ("logits", "in"):
                continue
            r = got[name]
            vals.append(sqnr_db(ref, (r["q"].astype(np.float64) - float(r["p"]["zero_point"])) * float(r["p"]["scale"])))
        return min(vals)

    # (a) the shortcut of the first residual add wired to the wrong tensor
    bad = [dict(o) for o in ops]
    bad[3]["b"] = "d1"
    assert worst_sqnr(netrun.run(bad, images, 2, SEED, 8)) < 15.0
    # (b) the add range taken from one input only: sums saturate
    monkeypatch.setattr(oracle, "add_output_range", lambda a, b, kind: oracle.range_after_activation(
        float(a["min_nudged"]), float(a["max_nudged"]), kind))
    assert worst_sqnr(netrun.run(ops, images, 2, SEED, 8)) < 30.0
    monkeypatch.undo()
    # (c) the bias dropped from the accumulators
    real_qb = oracle.quantize_bias
    monkeypatch.setattr(oracle, "quantize_bias", lambda b, xs, ws: np.zeros_like(real_qb(b, xs, ws)))
    assert worst_sqnr(netrun.run(ops, images, 2, SEED, 8)) < 30.0
    monkeypatch.undo()
    assert worst_sqnr(netrun.run(ops, images, 2, SEED, 8)) > 30.0
