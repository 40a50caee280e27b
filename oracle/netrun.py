"""Whole-network integer inference on the CPU oracle -- TEST INFRASTRUCTURE.

Post-training quantization as the paper describes it (Section 3.1.2): batch norm is folded into
the weights (Eq. 20-21), weights get per-channel symmetric quantizers from their min/max
(Sections 2.5-2.6), every activation tensor gets one affine quantizer from the range seen on a
calibration batch, and inference then runs in integers only (Eq. 4 + requantisation).

Organisation: one handler per op kind, looked up in `HANDLERS`; a handler receives the op record
and the tensors made so far and returns the op's output as a `QTensor` (codes + quantizer).  Every
arithmetic step is an `oracle` function; the range rules for the tensors between layers are
`oracle.range_after_activation` and `oracle.add_output_range` (qtz_oracle_net.c).  The layer list
and the random float parameters come from the shared shape module, which holds no arithmetic.

Readings that the paper leaves open: the input image codes 0..255 stand for reals in [0,1]
(scale 1/255, zero point 0); pooling keeps its input's quantizer; the classifier returns its
int32 accumulators.

Pins (tests/test_oracle_netrun.py): a float64 forward pass of the folded float network on a small
network (per-tensor SQNR, Appendix A), the range rules against closed forms, and the no-saturation
property of the add range.
"""
from __future__ import annotations

from typing import Callable, Dict, NamedTuple, Optional

import numpy as np

import oracle
from paper_1806_08342_b200 import synth


class QTensor(NamedTuple):
    q: np.ndarray                 # uint8 codes NHWC (int32 [B, classes] for the logits)
    p: Optional[np.void]          # quantizer record (None for the logits)


INPUT_SCALE = np.float32(1.0 / 255.0)


def input_quantizer():
    rec = np.zeros(1, oracle.QPARAMS)
    rec["scale"], rec["zero_point"], rec["min_nudged"], rec["max_nudged"] = INPUT_SCALE, 0, 0.0, 1.0
    return rec[0]


def quantized_weights(op, index, seed, wbits):
    """Folded and quantized weights of a conv / fc op: (integer codes, per-channel quantizers, float bias).
    Depthwise weights are HWC with the channel as the quantizer axis; dense weights OHWI with axis 0."""
    raw = synth.layer_params(op, index, seed)
    depthwise = bool(op.get("depthwise", False))
    w = raw["w"]
    if "bn" in raw:
        as_rows = np.ascontiguousarray(np.moveaxis(w, -1, 0)) if depthwise else w
        bn = raw["bn"]
        folded, bias = oracle.fold_batchnorm(as_rows, None, bn["gamma"], bn["beta"], bn["mean"], bn["var"], 1e-3)
        w = np.ascontiguousarray(np.moveaxis(folded, 0, -1)) if depthwise else folded
    else:
        bias = raw["bias"]
    channel_axis = w.ndim - 1 if depthwise else 0
    wq = oracle.calibrate_minmax(w, channel_axis, wbits, True)
    lo_code, hi_code = oracle.code_range(wbits, 1, 1 if wbits == 8 else 0)
    codes = oracle.quantize(w, wq, channel_axis, lo_code, hi_code)
    if wbits == 4:
        # the codes travel in packed form (two per byte along the reduction of an output channel, or along the
        # channels of a depthwise tap): take them through it so that the packing is part of what is checked
        rows = codes.reshape(-1, codes.shape[-1]) if depthwise else codes.reshape(codes.shape[0], -1)
        codes = oracle.unpack_s4(oracle.pack_s4(rows), rows.shape[1]).reshape(codes.shape)
    return codes, wq, bias


def output_quantizer(acc_calib, acc_scale, act):
    """Affine quantizer of a layer's output from the calibration accumulators (Section 2.5)."""
    per_channel = np.zeros(acc_calib.shape[-1], oracle.QPARAMS)
    per_channel["scale"] = acc_scale
    lo, hi = oracle.minmax(oracle.dequantize(acc_calib, per_channel, acc_calib.ndim - 1))
    lo, hi = oracle.range_after_activation(lo[0], hi[0], act)
    return oracle.affine_params(lo, hi, 8)


def _accumulate(op, x: QTensor, codes, bias_q):
    zx = int(x.p["zero_point"])
    if op["op"] == "fc":
        return oracle.conv2d_acc(x.q, zx, codes, None, bias_q, 1, 0)
    fn = oracle.depthwise_acc if op["depthwise"] else oracle.conv2d_acc
    return fn(x.q, zx, codes, None, bias_q, op["stride"], op["pad"])


def op_conv(op, index, t: Dict[str, QTensor], cfg) -> QTensor:
    x = t[op["src"]]
    x_scale = np.float32(x.p["scale"])
    codes, wq, bias = quantized_weights(op, index, cfg["seed"], cfg["wbits"])
    acc = _accumulate(op, x, codes, oracle.quantize_bias(bias, x_scale, wq["scale"]))
    if op["op"] == "fc":
        return QTensor(acc.reshape(acc.shape[0], -1), None)
    acc_scale = x_scale * wq["scale"]                      # fp32 product per output channel (Eq. 4: Delta_x Delta_w)
    yq = output_quantizer(acc[:cfg["calib"]], acc_scale, op["act"])
    pairs = [oracle.quantize_multiplier(float(x_scale) * float(s) / float(yq["scale"])) for s in wq["scale"]]
    mult = np.array([m for m, _ in pairs], np.int32)
    shift = np.array([r for _, r in pairs], np.int32)
    lo_code, hi_code = oracle.activation_range(op["act"], yq["scale"], int(yq["zero_point"]))
    y = oracle.requantize(acc, mult, shift, int(yq["zero_point"]), lo_code, hi_code)
    return QTensor(y.astype(np.uint8), yq)


def op_add(op, index, t, cfg) -> QTensor:
    a, b = t[op["a"]], t[op["b"]]
    lo, hi = oracle.add_output_range(a.p, b.p, op["act"])
    yq = oracle.affine_params(lo, hi, 8)
    m_a, m_b, shift = oracle.add_params(a.p["scale"], b.p["scale"], yq["scale"])
    lo_code, hi_code = oracle.activation_range(op["act"], yq["scale"], int(yq["zero_point"]))
    y = oracle.add_u8(a.q, int(a.p["zero_point"]), m_a, b.q, int(b.p["zero_point"]), m_b, shift,
                      int(yq["zero_point"]), lo_code, hi_code)
    return QTensor(y, yq)


def op_maxpool(op, index, t, cfg) -> QTensor:
    x = t[op["src"]]
    return QTensor(oracle.maxpool_u8(x.q, op["k"], op["stride"], op["pad"]), x.p)


def op_avgpool(op, index, t, cfg) -> QTensor:
    x = t[op["src"]]
    pixels = x.q.shape[1] * x.q.shape[2]
    mult, shift = oracle.quantize_multiplier(1.0 / pixels)       # same quantizer in and out: M = 1 / (H W)
    z = int(x.p["zero_point"])
    return QTensor(oracle.global_avgpool_u8(x.q, z, mult, shift, z), x.p)


HANDLERS: Dict[str, Callable] = {"conv": op_conv, "fc": op_conv, "add": op_add, "maxpool": op_maxpool,
                                 "avgpool": op_avgpool}


def run(ops, images, calib, seed, wbits=8, visit=None, keep=True):
    """Runs `ops` on uint8 `images` [B,H,W,3]; activation ranges come from images[:calib].
    Returns {tensor name: {"q": codes, "p": quantizer record}}; "logits" holds int32 [B, classes].
    `visit(name, QTensor)` is called for every tensor as it is made; with keep=False tensors are dropped
    once no later op reads them (whole batches of the large networks) and only the logits are returned."""
    cfg = {"calib": calib, "seed": seed, "wbits": wbits}
    last_use = {}
    for i, op in enumerate(ops):
        for key in ("src", "a", "b"):
            if key in op:
                last_use[op[key]] = i
    t: Dict[str, QTensor] = {"in": QTensor(images, input_quantizer())}
    if visit:
        visit("in", t["in"])
    for index, op in enumerate(ops):
        out = HANDLERS[op["op"]](op, index, t, cfg)
        t[op["dst"]] = out
        if visit:
            visit(op["dst"], out)
        if not keep:
            for name in [n for n, last in last_use.items() if last == index and n in t]:
                del t[name]
    return {name: {"q": v.q, "p": v.p} for name, v in t.items()}
