"""CPU oracle for integer-only quantized convolution -- TEST INFRASTRUCTURE.

Thin numpy marshalling around the plain-C oracle in this directory
(``qtz_oracle*.c``).  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; it shares nothing with the CUDA
library and is never a fallback for it.

All arithmetic lives in the C files, each function citing the passage of the
paper it follows.  This module only reshapes arrays and calls them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SOURCES = ["qtz_oracle.c", "qtz_oracle_conv.c", "qtz_oracle_ops.c", "qtz_oracle_sim.c", "qtz_oracle_net.c", "qtz_oracle_act4.c"]
_LIB_PATH = os.path.join(_DIR, "liboracle.so")
_lib = None

QPARAMS = np.dtype([("scale", "<f4"), ("zero_point", "<i4"),
                    ("min_nudged", "<f4"), ("max_nudged", "<f4")])


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    srcs = [os.path.join(_DIR, s) for s in _SOURCES]
    deps = srcs + [os.path.join(_DIR, "orc_common.h")]
    if (not force and os.path.exists(_LIB_PATH)
            and all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in deps)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
           "-shared", "-fPIC", "-o", _LIB_PATH] + srcs + ["-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle use."""
    return int(lib().orc_set_threads(0))


def set_num_threads(n: int) -> int:
    """Sets the number of OpenMP threads (timing runs); returns the value now in force."""
    return int(lib().orc_set_threads(int(n)))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _chk(rc):
    if rc != 0:
        raise OracleError(rc)


def _view(shape, axis):
    if axis is None:
        return 1, 1, int(np.prod(shape, dtype=np.int64))
    axis = axis % len(shape)
    return (int(np.prod(shape[:axis], dtype=np.int64)), int(shape[axis]),
            int(np.prod(shape[axis + 1:], dtype=np.int64)))


I64, I32, F32 = ctypes.c_int64, ctypes.c_int32, ctypes.c_float


def minmax(x, axis=None):
    x = np.ascontiguousarray(x, dtype=np.float32)
    o, a, i = _view(x.shape, axis)
    lo = np.empty(a, np.float32)
    hi = np.empty(a, np.float32)
    _chk(lib().orc_minmax(_p(x), I64(o), I64(a), I64(i), _p(lo), _p(hi)))
    return lo, hi


def affine_params(lo, hi, bits=8):
    q = np.zeros(1, QPARAMS)
    _chk(lib().orc_affine_params(F32(lo), F32(hi), int(bits), _p(q)))
    return q[0]


def symmetric_params(lo, hi, bits=8):
    q = np.zeros(1, QPARAMS)
    _chk(lib().orc_symmetric_params(F32(lo), F32(hi), int(bits), _p(q)))
    return q[0]


def calibrate_minmax(x, axis=None, bits=8, symmetric=False):
    x = np.ascontiguousarray(x, dtype=np.float32)
    o, a, i = _view(x.shape, axis)
    q = np.zeros(a, QPARAMS)
    _chk(lib().orc_calibrate_minmax(_p(x), I64(o), I64(a), I64(i), int(bits),
                                    int(bool(symmetric)), _p(q)))
    return q


def code_range(bits, is_signed, restrict_range):
    lo, hi = I32(), I32()
    _chk(lib().orc_code_range(int(bits), int(is_signed), int(restrict_range),
                              ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value


def quantize(x, params, axis, qmin, qmax):
    x = np.ascontiguousarray(x, dtype=np.float32)
    params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
    o, a, i = _view(x.shape, axis)
    assert params.shape[0] == a
    q = np.empty(x.shape, np.int32)
    _chk(lib().orc_quantize(_p(x), I64(o), I64(a), I64(i), _p(params), I32(qmin), I32(qmax),
                            _p(q)))
    return q


def dequantize(q, params, axis):
    q = np.ascontiguousarray(q, dtype=np.int32)
    params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
    o, a, i = _view(q.shape, axis)
    assert params.shape[0] == a
    x = np.empty(q.shape, np.float32)
    _chk(lib().orc_dequantize(_p(q), I64(o), I64(a), I64(i), _p(params), _p(x)))
    return x


def pack_s4(codes):
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    k = codes.shape[-1]
    rows = codes.size // k
    out = np.empty(codes.shape[:-1] + ((k + 1) // 2,), np.uint8)
    _chk(lib().orc_pack_s4(_p(codes), I64(rows), I64(k), _p(out)))
    return out


def unpack_s4(packed, k):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    rows = packed.size // packed.shape[-1]
    out = np.empty(packed.shape[:-1] + (k,), np.int32)
    _chk(lib().orc_unpack_s4(_p(packed), I64(rows), I64(k), _p(out)))
    return out


def fold_batchnorm(w, conv_bias, gamma, beta, mean, var, eps):
    w = np.ascontiguousarray(w, dtype=np.float32)
    n = w.shape[0]
    k = w.size // n
    f = lambda v: None if v is None else np.ascontiguousarray(v, dtype=np.float32)
    cb, g, b, m, v = f(conv_bias), f(gamma), f(beta), f(mean), f(var)
    w_inf = np.empty_like(w)
    bias_inf = np.empty(n, np.float32)
    _chk(lib().orc_fold_batchnorm(_p(w), _p(cb), _p(g), _p(b), _p(m), _p(v), F32(eps),
                                  I64(n), I64(k), _p(w_inf), _p(bias_inf)))
    return w_inf, bias_inf


def quantize_bias(bias, x_scale, w_scale):
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    out = np.empty(bias.shape[0], np.int32)
    _chk(lib().orc_quantize_bias(_p(bias), I64(bias.shape[0]), F32(x_scale), _p(w_scale),
                                 _p(out)))
    return out


def quantize_multiplier(real_multiplier):
    m, r = I32(), I32()
    _chk(lib().orc_quantize_multiplier(ctypes.c_double(real_multiplier), ctypes.byref(m),
                                       ctypes.byref(r)))
    return m.value, r.value


def activation_range(kind, y_scale, y_zero_point):
    lo, hi = I32(), I32()
    _chk(lib().orc_activation_range(int(kind), F32(y_scale), I32(y_zero_point),
                                    ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value


def requantize(acc, mult, rshift, y_zero_point, act_min=0, act_max=255):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    n = acc.shape[-1]
    mult = np.ascontiguousarray(mult, dtype=np.int32)
    rshift = np.ascontiguousarray(rshift, dtype=np.int32)
    assert mult.shape == (n,) and rshift.shape == (n,)
    y = np.empty(acc.shape, np.int32)
    _chk(lib().orc_requantize(_p(acc), I64(acc.size // n), I64(n), _p(mult), _p(rshift),
                              I32(y_zero_point), I32(act_min), I32(act_max), _p(y)))
    return y


def _conv_common(x, c, w, z_w, bias_q):
    x = np.ascontiguousarray(x, dtype=np.uint8)
    assert x.ndim == 4
    w = np.ascontiguousarray(w, dtype=np.int32)
    zw = None if z_w is None else np.ascontiguousarray(z_w, dtype=np.int32)
    bq = None if bias_q is None else np.ascontiguousarray(bias_q, dtype=np.int32)
    return x, w, zw, bq


def conv2d_acc(x, z_x, w, z_w=None, bias_q=None, stride=1, pad=0, c=None, expanded=False):
    """x: uint8 [B,H,W,pitch] (first c channels used); w: int codes [N,KH,KW,C];
    z_w: None or int32[N].  Returns int32 accumulators [B,OH,OW,N]."""
    x, w, zw, bq = _conv_common(x, c, w, z_w, bias_q)
    b, h, ww, xp = x.shape
    n, kh, kw, cc = w.shape
    c = cc if c is None else c
    assert c == cc and xp >= c
    if zw is not None:
        assert zw.shape == (n,)
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (ww + 2 * pad - kw) // stride + 1
    acc = np.empty((b, oh, ow, n), np.int32)
    fn = lib().orc_conv2d_acc_expanded if expanded else lib().orc_conv2d_acc
    _chk(fn(_p(x), I32(b), I32(h), I32(ww), I32(c), I32(xp), I32(z_x), _p(w), _p(zw), _p(bq),
            I32(n), I32(kh), I32(kw), I32(stride), I32(pad), _p(acc)))
    return acc


def depthwise_acc(x, z_x, w, z_w=None, bias_q=None, stride=1, pad=1, c=None):
    """x: uint8 [B,H,W,pitch]; w: int codes [KH,KW,C].  Returns int32 [B,OH,OW,C]."""
    x, w, zw, bq = _conv_common(x, c, w, z_w, bias_q)
    b, h, ww, xp = x.shape
    kh, kw, cc = w.shape
    c = cc if c is None else c
    assert c == cc and xp >= c
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (ww + 2 * pad - kw) // stride + 1
    acc = np.empty((b, oh, ow, c), np.int32)
    _chk(lib().orc_depthwise_acc(_p(x), I32(b), I32(h), I32(ww), I32(c), I32(xp), I32(z_x),
                                 _p(w), _p(zw), _p(bq), I32(kh), I32(kw), I32(stride),
                                 I32(pad), _p(acc)))
    return acc


def add_params(a_scale, b_scale, y_scale):
    ma, mb, r = I32(), I32(), I32()
    _chk(lib().orc_add_params(F32(a_scale), F32(b_scale), F32(y_scale), ctypes.byref(ma),
                              ctypes.byref(mb), ctypes.byref(r)))
    return ma.value, mb.value, r.value


def add_u8(a, z_a, m_a, b, z_b, m_b, rshift, z_y, act_min, act_max, c=None):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    b = np.ascontiguousarray(b, dtype=np.uint8)
    assert a.shape == b.shape
    pitch = a.shape[-1]
    c = pitch if c is None else c
    y = np.zeros_like(a)
    _chk(lib().orc_add_u8(_p(a), I32(z_a), I32(m_a), _p(b), I32(z_b), I32(m_b), I32(rshift),
                          I32(z_y), I32(act_min), I32(act_max), I64(a.size // pitch), I32(c),
                          I32(pitch), _p(y)))
    return y


def maxpool_u8(x, k, stride, pad, c=None):
    x = np.ascontiguousarray(x, dtype=np.uint8)
    b, h, w, xp = x.shape
    c = xp if c is None else c
    oh = (h + 2 * pad - k) // stride + 1
    ow = (w + 2 * pad - k) // stride + 1
    y = np.zeros((b, oh, ow, xp), np.uint8)
    _chk(lib().orc_maxpool_u8(_p(x), I32(b), I32(h), I32(w), I32(c), I32(xp), I32(k),
                              I32(stride), I32(pad), I32(xp), _p(y)))
    return y


def global_avgpool_u8(x, z_x, mult, rshift, z_y, c=None):
    x = np.ascontiguousarray(x, dtype=np.uint8)
    b, h, w, xp = x.shape
    c = xp if c is None else c
    y = np.zeros((b, 1, 1, xp), np.uint8)
    _chk(lib().orc_global_avgpool_u8(_p(x), I32(z_x), I32(b), I32(h * w), I32(c), I32(xp),
                                     I32(mult), I32(rshift), I32(z_y), I32(xp), _p(y)))
    return y


def simquant(x, params, axis, qmin, qmax):
    """SimQuant (Section 2.4): quantize then de-quantize, fp32 in and out."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
    o, a, i = _view(x.shape, axis)
    assert params.shape[0] == a
    y = np.empty(x.shape, np.float32)
    _chk(lib().orc_simquant(_p(x), I64(o), I64(a), I64(i), _p(params), I32(qmin), I32(qmax), _p(y)))
    return y


def sqnr(w, w_hat, axis=None):
    """SQNR in dB (Appendix A) per index of `axis`, or of the whole tensor (axis=None)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    w_hat = np.ascontiguousarray(w_hat, dtype=np.float32)
    assert w.shape == w_hat.shape
    o, a, i = _view(w.shape, axis)
    out = np.empty(a, np.float64)
    _chk(lib().orc_sqnr(_p(w), _p(w_hat), I64(o), I64(a), I64(i), _p(out)))
    return out


def ema_update(state_lo, state_hi, batch_lo, batch_hi, decay, initialised):
    """Moving average of per-batch ranges (Section 2.5); updates the fp64 state arrays in place and
    returns the new `initialised` flag."""
    assert state_lo.dtype == np.float64 and state_hi.dtype == np.float64
    batch_lo = np.ascontiguousarray(batch_lo, dtype=np.float32)
    batch_hi = np.ascontiguousarray(batch_hi, dtype=np.float32)
    flag = I32(int(bool(initialised)))
    _chk(lib().orc_ema_update(_p(state_lo), _p(state_hi), _p(batch_lo), _p(batch_hi), I64(state_lo.size),
                              ctypes.c_double(decay), ctypes.byref(flag)))
    return bool(flag.value)


def rescale_u8(x, z_x, mult, rshift, z_y, act_min=0, act_max=255, c=None, out=None, out_offset=0):
    """uint8 tensor to another quantizer (concat, Section 3.2.1).  x: [..., pitch]; the result goes to
    `out[..., out_offset:out_offset + c]` when `out` is given (a channel slice of a concatenation)."""
    x = np.ascontiguousarray(x, dtype=np.uint8)
    xp = x.shape[-1]
    c = xp if c is None else c
    if out is None:
        out = np.zeros_like(x)
    assert out.flags["C_CONTIGUOUS"] and out.dtype == np.uint8
    yp = out.shape[-1]
    dst = ctypes.c_void_p(out.ctypes.data + out_offset)
    _chk(lib().orc_rescale_u8(_p(x), I64(x.size // xp), I32(c), I32(xp), I32(z_x), I32(mult), I32(rshift),
                              I32(z_y), I32(act_min), I32(act_max), dst, I32(yp)))
    return out


def range_after_activation(lo, hi, kind):
    """Observed pre-activation range pushed through the fused activation (0 none, 1 ReLU, 2 ReLU6)."""
    a, b = F32(), F32()
    _chk(lib().orc_range_after_activation(F32(lo), F32(hi), I32(kind), ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def add_output_range(a_params, b_params, kind):
    """Range of a + b from the inputs' nudged ranges, then the fused activation."""
    pa = np.ascontiguousarray(np.atleast_1d(a_params), dtype=QPARAMS)
    pb = np.ascontiguousarray(np.atleast_1d(b_params), dtype=QPARAMS)
    lo, hi = F32(), F32()
    _chk(lib().orc_add_output_range(_p(pa), _p(pb), I32(kind), ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value


def pack_u4(codes, packed_pitch=None):
    """Unsigned 4-bit activation codes [..., k] (uint8, values 0..15) -> two per byte along k."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    k = codes.shape[-1]
    pitch = (k + 1) // 2 if packed_pitch is None else packed_pitch
    out = np.zeros(codes.shape[:-1] + (pitch,), np.uint8)
    _chk(lib().orc_pack_u4(_p(codes), I64(codes.size // k), I64(k), I64(k), _p(out), I64(pitch)))
    return out


def unpack_u4(packed, k):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    pitch = packed.shape[-1]
    out = np.zeros(packed.shape[:-1] + (k,), np.uint8)
    _chk(lib().orc_unpack_u4(_p(packed), I64(packed.size // pitch), I64(k), I64(pitch), _p(out), I64(k)))
    return out


def activation_range_bits(kind, y_scale, y_zero_point, bits):
    lo, hi = I32(), I32()
    _chk(lib().orc_activation_range_bits(int(kind), F32(y_scale), I32(y_zero_point), int(bits),
                                         ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value
