"""Whole-network integer inference on the CPU oracle -- TEST INFRASTRUCTURE.

Post-training quantization as the paper describes it (Section 3.1.2): batch norm is folded into
the weights (Eq. 20-21), weights get per-channel symmetric quantizers from their min/max
(Section 2.5-2.6), every activation tensor gets one affine quantizer from the min/max seen on a
calibration batch, and inference then runs in integers only (Eq. 4 + requantisation).
Only `oracle` functions do arithmetic here; the layer list comes from the shared shape module.

Readings that the paper leaves open: the input image codes 0..255 stand for reals in [0,1]
(scale 1/255, zero point 0); the range of a layer followed by ReLU / ReLU6 is the min/max of its
real outputs clamped to [0,inf) / [0,6]; the range of a residual add is the sum of its inputs'
nudged ranges (a bound, not a measurement); pooling keeps its input's quantizer.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_1806_08342_b200 import synth


def _record(scale, zp, lo, hi):
    q = np.zeros(1, oracle.QPARAMS)
    q["scale"], q["zero_point"], q["min_nudged"], q["max_nudged"] = scale, zp, lo, hi
    return q[0]


def _weights(op, index, seed, wbits):
    """Folded, quantized weights of a conv / fc op: (codes, per-channel params, float bias)."""
    p = synth.layer_params(op, index, seed)
    w = p["w"]
    depthwise = op["op"] == "conv" and op["depthwise"]
    if "bn" in p:
        bn = p["bn"]
        rows = np.ascontiguousarray(np.moveaxis(w, 2, 0)) if depthwise else w        # one row per output channel
        rows, bias = oracle.fold_batchnorm(rows, None, bn["gamma"], bn["beta"], bn["mean"], bn["var"], 1e-3)
        w = np.ascontiguousarray(np.moveaxis(rows, 0, 2)) if depthwise else rows
    else:
        bias = p["bias"]
    axis = 2 if depthwise else 0
    wp = oracle.calibrate_minmax(w, axis, wbits, True)
    qmin, qmax = oracle.code_range(wbits, 1, 1 if wbits == 8 else 0)
    codes = oracle.quantize(w, wp, axis, qmin, qmax)
    if wbits == 4:                                                                    # through the packed form and back
        flat = codes.reshape(9, -1) if depthwise else codes.reshape(codes.shape[0], -1)
        codes = oracle.unpack_s4(oracle.pack_s4(flat), flat.shape[1]).reshape(codes.shape)
    return codes, wp, bias


def run(ops, images, calib, seed, wbits=8):
    """Runs `ops` on uint8 `images` [B,H,W,3]; activation ranges come from images[:calib].
    Returns {tensor name: {"q": codes, "p": qparams record}}; "logits" holds int32 [B, classes]."""
    t = {"in": {"q": images, "p": _record(np.float32(1.0 / 255.0), 0, np.float32(0.0), np.float32(1.0))}}
    for index, op in enumerate(ops):
        kind = op["op"]
        if kind in ("conv", "fc"):
            x = t[op["src"]]
            xs, zx = np.float32(x["p"]["scale"]), int(x["p"]["zero_point"])
            codes, wp, bias = _weights(op, index, seed, wbits)
            bq = oracle.quantize_bias(bias, xs, wp["scale"])
            if kind == "fc":
                acc = oracle.conv2d_acc(x["q"], zx, codes, None, bq, 1, 0)
                t[op["dst"]] = {"q": acc.reshape(acc.shape[0], -1), "p": None}
                continue
            if op["depthwise"]:
                acc = oracle.depthwise_acc(x["q"], zx, codes, None, bq, op["stride"], op["pad"])
            else:
                acc = oracle.conv2d_acc(x["q"], zx, codes, None, bq, op["stride"], op["pad"])
            ap = np.zeros(acc.shape[-1], oracle.QPARAMS)
            ap["scale"] = xs * wp["scale"]                                            # fp32 product, formed once
            lo, hi = oracle.minmax(oracle.dequantize(acc[:calib], ap, 3))
            lo, hi = float(lo[0]), float(hi[0])
            if op["act"] == 1:
                lo, hi = max(lo, 0.0), max(hi, 0.0)
            elif op["act"] == 2:
                lo, hi = min(max(lo, 0.0), 6.0), min(max(hi, 0.0), 6.0)
            yp = oracle.affine_params(lo, hi, 8)
            mr = [oracle.quantize_multiplier(float(xs) * float(s) / float(yp["scale"])) for s in wp["scale"]]
            amin, amax = oracle.activation_range(op["act"], yp["scale"], int(yp["zero_point"]))
            y = oracle.requantize(acc, np.array([m for m, _ in mr], np.int32), np.array([r for _, r in mr], np.int32),
                                  int(yp["zero_point"]), amin, amax)
            t[op["dst"]] = {"q": y.astype(np.uint8), "p": yp}
        elif kind == "add":
            a, b = t[op["a"]], t[op["b"]]
            lo = float(np.float32(a["p"]["min_nudged"]) + np.float32(b["p"]["min_nudged"]))
            hi = float(np.float32(a["p"]["max_nudged"]) + np.float32(b["p"]["max_nudged"]))
            if op["act"] == 1:
                lo, hi = max(lo, 0.0), max(hi, 0.0)
            yp = oracle.affine_params(lo, hi, 8)
            ma, mb, r = oracle.add_params(a["p"]["scale"], b["p"]["scale"], yp["scale"])
            amin, amax = oracle.activation_range(op["act"], yp["scale"], int(yp["zero_point"]))
            y = oracle.add_u8(a["q"], int(a["p"]["zero_point"]), ma, b["q"], int(b["p"]["zero_point"]), mb, r,
                              int(yp["zero_point"]), amin, amax)
            t[op["dst"]] = {"q": y, "p": yp}
        elif kind == "maxpool":
            x = t[op["src"]]
            t[op["dst"]] = {"q": oracle.maxpool_u8(x["q"], op["k"], op["stride"], op["pad"]), "p": x["p"]}
        elif kind == "avgpool":
            x = t[op["src"]]
            hw = x["q"].shape[1] * x["q"].shape[2]
            m, r = oracle.quantize_multiplier(1.0 / hw)
            z = int(x["p"]["zero_point"])
            t[op["dst"]] = {"q": oracle.global_avgpool_u8(x["q"], z, m, r, z), "p": x["p"]}
        else:
            raise ValueError(kind)
    return t
