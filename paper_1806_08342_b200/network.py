"""Whole-network integer inference through libqtz (MobileNet-v1/v2, ResNet-50 shapes).

Every numerical step is a call into the C ABI (`qtz.py`): batch-norm folding, weight and
activation calibration, quantization, the convolutions, the residual adds and the pooling all run
in the library's CUDA kernels.  This module only sequences the calls and keeps the tensors.

`QuantizedNetwork.build()` performs post-training quantization on a calibration batch (Section
3.1.2 of the paper: ranges of activations from calibration data, per-channel weight quantizers);
`QuantizedNetwork.forward()` is the integer-only inference pass that the benchmark times.
"""
from __future__ import annotations

import numpy as np
import torch

from . import qtz, synth


def _rup16(v):
    return (v + 15) // 16 * 16


class _Layer:
    __slots__ = ("op", "plan", "args", "out_shape", "out_c", "out_params")


class QuantizedNetwork:
    def __init__(self, handle: qtz.Handle, ops, seed: int, wbits: int = 8, fuse: bool = True, fuse_depthwise: bool = False):
        self.h, self.ops, self.seed, self.wbits = handle, ops, seed, wbits
        self.fuse = fuse            # forward() runs a convolution and the residual add that follows it as one kernel
        # forward() runs a 3x3 depthwise layer and the pointwise layer after it as one kernel where the library can
        # (qtz_conv2d_dw_pw_u8).  Off by default: on the networks here the two separate kernels are faster.
        self.fuse_depthwise = fuse_depthwise
        self.fused_away = set()     # tensors forward() then never writes (build() still computes them once)
        self.schedule = []          # what forward() launches: (kind, layer[, add layer])
        self.layers = []
        self.params = {}            # tensor name -> qparams record (numpy void) after build()
        self.batch = None

    # ---- weights ---------------------------------------------------------------------------
    def _prepare_weights(self, op, index, x_scale):
        """Folds, calibrates and quantizes the weights of one conv / fc op on the device.
        Returns (w_q tensor in API layout, per-channel params, int32 bias tensor, wkind)."""
        h = self.h
        p = synth.layer_params(op, index, self.seed)
        depthwise = op["op"] == "conv" and op["depthwise"]
        w = torch.from_numpy(p["w"]).cuda()
        if "bn" in p:
            bn = {k: torch.from_numpy(v).cuda() for k, v in p["bn"].items()}
            rows = w.permute(2, 0, 1).contiguous() if depthwise else w          # one row per output channel
            rows, bias = h.fold_batchnorm(rows, None, bn["gamma"], bn["beta"], bn["mean"], bn["var"], 1e-3)
            w = rows.permute(1, 2, 0).contiguous() if depthwise else rows
        else:
            bias = torch.from_numpy(p["bias"]).cuda()
        axis = 2 if depthwise else 0
        wp = h.calibrate_minmax(w, axis=axis, bits=self.wbits, symmetric=True)
        if self.wbits == 8:
            w_q = h.quantize_tensor(w, wp, axis=axis, out_dtype=qtz.S8, restrict_range=True)
            wkind = qtz.W_S8_PER_CHANNEL_SYM
        else:
            # packed 4-bit: along k of each output channel (dense) or along the channels of each tap (depthwise)
            flat = w.reshape(9, -1) if depthwise else w.reshape(w.shape[0], -1)
            w_q = h.quantize_tensor(flat, wp, axis=1 if depthwise else 0, out_dtype=qtz.S4_PACKED)
            wkind = qtz.W_S4_PACKED_PER_CHANNEL_SYM
        bias_q = h.quantize_bias(bias, x_scale, wp)
        return w_q, wp, bias_q, wkind

    # ---- calibration + plan creation -------------------------------------------------------
    def build(self, images_u8: np.ndarray, calib: int):
        """images_u8: [B,H,W,3].  Calibrates on images[:calib], creates plans for batch B and runs
        the whole batch once.  Returns {tensor name: device tensor}."""
        h = self.h
        batch = images_u8.shape[0]
        self.batch = batch
        x0 = np.zeros(images_u8.shape[:3] + (4,), np.uint8)          # images at 4 bytes per pixel (the stem repacks them)
        x0[..., :3] = images_u8
        tensors = {"in": torch.from_numpy(x0).cuda()}
        chans = {"in": 3}
        self.params = {"in": qtz.params_from_range(0.0, 1.0)}   # image codes 0..255 stand for reals in [0,1]
        self.layers = []
        for index, op in enumerate(self.ops):
            kind = op["op"]
            L = _Layer()
            L.op = op
            if kind in ("conv", "fc"):
                x, xp = tensors[op["src"]], self.params[op["src"]]
                xs, zx = np.float32(xp["scale"]), int(xp["zero_point"])
                w_q, wp, bias_q, wkind = self._prepare_weights(op, index, xs)
                _, hh, ww, pitch = x.shape
                k, st, pad = (1, 1, 0) if kind == "fc" else (op["k"], op["stride"], op["pad"])
                cin, cout = op["cin"], op["cout"]
                dw = kind == "conv" and op["depthwise"]
                raw_desc = qtz.conv_desc(calib if kind == "conv" else batch, hh, ww, cin, cout, k, k, st, pad, wkind,
                                         qtz.OUT_S32_RAW, c_pitch_in=pitch)
                raw_plan = h.conv_create(raw_desc, w_q, bias_q, depthwise=dw)
                if kind == "fc":
                    L.plan, L.args = raw_plan, (zx,)
                    tensors[op["dst"]] = raw_plan(x, zx).reshape(batch, cout)
                    self.params[op["dst"]] = None
                    self.layers.append(L)
                    continue
                acc = raw_plan(x[:calib], zx)
                lo, hi = h.minmax(h.dequantize(acc, qtz.accumulator_scales(xs, wp), axis=3))
                raw_plan.close()
                yp = qtz.params_from_range(*qtz.range_after_activation(lo[0], hi[0], op["act"]))
                mult, rshift = qtz.requant_multipliers(xs, wp, yp["scale"])
                amin, amax = qtz.activation_range(op["act"], yp["scale"], int(yp["zero_point"]))
                desc = qtz.conv_desc(batch, hh, ww, cin, cout, k, k, st, pad, wkind, qtz.OUT_U8, c_pitch_in=pitch)
                L.plan = h.conv_create(desc, w_q, bias_q, None, mult, rshift, depthwise=dw)
                L.args = (zx, int(yp["zero_point"]), amin, amax)
                tensors[op["dst"]] = L.plan(x, *L.args)
                chans[op["dst"]] = cout
                self.params[op["dst"]] = yp
            elif kind == "add":
                a, b = self.params[op["a"]], self.params[op["b"]]
                yp = qtz.params_from_range(*qtz.add_output_range(a, b, op["act"]))
                ma, mb, r = qtz.add_params(a["scale"], b["scale"], yp["scale"])
                amin, amax = qtz.activation_range(op["act"], yp["scale"], int(yp["zero_point"]))
                L.args = (int(a["zero_point"]), ma, int(b["zero_point"]), mb, r, int(yp["zero_point"]), amin, amax,
                          chans[op["a"]])
                ta, tb = tensors[op["a"]], tensors[op["b"]]
                tensors[op["dst"]] = h.add_u8(ta, L.args[0], ma, tb, L.args[2], mb, r, *L.args[5:])
                chans[op["dst"]] = chans[op["a"]]
                self.params[op["dst"]] = yp
            elif kind == "maxpool":
                x = tensors[op["src"]]
                L.args = (chans[op["src"]], op["k"], op["stride"], op["pad"])
                tensors[op["dst"]] = h.maxpool_u8(x, *L.args)
                chans[op["dst"]] = chans[op["src"]]
                self.params[op["dst"]] = self.params[op["src"]]
            elif kind == "avgpool":
                x, xp = tensors[op["src"]], self.params[op["src"]]
                m, r = qtz.avgpool_multiplier(x.shape[1] * x.shape[2], xp["scale"], xp["scale"])
                z = int(xp["zero_point"])
                L.args = (z, z, m, r, chans[op["src"]])
                tensors[op["dst"]] = h.global_avgpool_u8(x, *L.args)
                chans[op["dst"]] = chans[op["src"]]
                self.params[op["dst"]] = xp
            else:
                raise ValueError(kind)
            self.layers.append(L)
        self.tensors = tensors
        self.chans = chans
        self._plan_schedule()
        return tensors

    def _plan_schedule(self):
        """Pairs every element-wise add with the convolution that produces one of its inputs, when that tensor has no
        other reader and the convolution runs on the tensor-core path: the pair becomes one qtz_conv2d_add_u8 call
        at the add's position (Section 3.2.1: the add fuses into the producing op)."""
        readers = {}
        for L in self.layers:
            for key in ("src", "a", "b"):
                if key in L.op:
                    readers[L.op[key]] = readers.get(L.op[key], 0) + 1
        producer = {L.op["dst"]: L for L in self.layers}
        taken, fused = set(), {}
        if self.fuse:
            for L in self.layers:
                if L.op["op"] != "add":
                    continue
                for mine, other in (("a", "b"), ("b", "a")):
                    P = producer.get(L.op[mine])
                    if (P is not None and P.op["op"] == "conv" and not P.op["depthwise"] and P.plan.kernel == "tcgen05"
                            and readers.get(L.op[mine], 0) == 1 and id(P) not in taken):
                        taken.add(id(P))
                        fused[id(L)] = (P, mine, other)
                        break
        self.fused_away = {P.op["dst"] for P, _, _ in fused.values()}
        # depthwise -> pointwise pairs: the depthwise output has the pointwise layer as its only reader; the library
        # decides whether the pair can run as one kernel (a first call here, into the pointwise layer's own output)
        blocks = {}
        if self.fuse_depthwise:
            t = self.tensors
            for D in self.layers:
                if D.op["op"] != "conv" or not D.op["depthwise"] or readers.get(D.op["dst"], 0) != 1:
                    continue
                P = next((L for L in self.layers if L.op.get("src") == D.op["dst"]), None)
                if (P is None or P.op["op"] != "conv" or P.op["depthwise"] or P.op["k"] != 1 or P.op["stride"] != 1
                        or id(P) in taken or P.plan.kernel != "tcgen05"):
                    continue
                try:
                    P.plan.after_depthwise(D.plan, t[D.op["src"]], *D.args, *P.args[1:], out=t[P.op["dst"]])
                except qtz.QtzError as e:
                    if e.code != -3:        # QTZ_ERR_UNSUPPORTED: the pair stays two kernels
                        raise
                    continue
                blocks[id(P)] = D
                taken.add(id(D))
                self.fused_away.add(D.op["dst"])
        self.schedule = []
        for L in self.layers:
            if id(L) in taken:
                continue
            if id(L) in blocks:
                self.schedule.append(("dw+pw", L, blocks[id(L)]))
            elif id(L) in fused:
                P, mine, other = fused[id(L)]
                a = L.args      # (za, ma, zb, mb, r, zy, amin, amax, c)
                t_zp, t_mult, s_zp, s_mult = (a[0], a[1], a[2], a[3]) if mine == "a" else (a[2], a[3], a[0], a[1])
                res = qtz.Residual(t_zp, P.args[2], P.args[3], t_mult, s_zp, s_mult, a[4])
                self.schedule.append(("conv+add", P, L, res, other))
            else:
                self.schedule.append((L.op["op"], L))

    # ---- the timed pass ----------------------------------------------------------------------
    def forward(self, x=None):
        """Integer-only inference of the whole batch with the plans made by build(); writes into the
        tensors build() allocated.  Returns the int32 logits tensor."""
        h, t = self.h, self.tensors
        if x is not None:
            t["in"] = x
        for item in self.schedule:
            self.run_item(item)
        return t["logits"]

    def run_item(self, item):
        """One entry of the schedule: a library call on the tensors build() allocated."""
        h, t = self.h, self.tensors
        kind, L = item[0], item[1]
        op = L.op
        if kind == "conv+add":
            _, P, A, res, other = item
            a = A.args
            P.plan.add_fused(t[P.op["src"]], P.args[0], res, t[A.op[other]], a[5], a[6], a[7], out=t[A.op["dst"]])
        elif kind == "dw+pw":
            D = item[2]
            L.plan.after_depthwise(D.plan, t[D.op["src"]], *D.args, *L.args[1:], out=t[op["dst"]])
        elif kind in ("conv", "fc"):
            L.plan(t[op["src"]], *L.args, out=t[op["dst"]])
        elif kind == "add":
            a = L.args
            h.add_u8(t[op["a"]], a[0], a[1], t[op["b"]], a[2], a[3], a[4], a[5], a[6], a[7], a[8], out=t[op["dst"]])
        elif kind == "maxpool":
            h.maxpool_u8(t[op["src"]], *L.args, out=t[op["dst"]])
        else:
            h.global_avgpool_u8(t[op["src"]], *L.args, out=t[op["dst"]])

    def num_launch_calls(self):
        return len(self.schedule)
