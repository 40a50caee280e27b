"""ctypes binding of libqtz (the C ABI in ``include/qtz.h``).

Argument marshalling only: every function takes torch CUDA tensors (PyTorch is used
for device memory and streams), passes their pointers and sizes to the entry point of
the same name, and raises :class:`QtzError` on a non-zero status.  There is no
fallback: if ``libqtz.so`` has not been built this module raises on first use.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int32, c_int64, c_void_p

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libqtz.so")

U8, S8, S4_PACKED, S32, U4_PACKED, U16, S16 = 0, 1, 2, 3, 4, 5, 6
W_S8_PER_CHANNEL_SYM, W_U8_PER_LAYER_ASYM, W_S4_PACKED_PER_CHANNEL_SYM = 0, 1, 2
OUT_U8, OUT_S32_RAW = 0, 1
ACT_NONE, ACT_RELU, ACT_RELU6 = 0, 1, 2

QPARAMS = np.dtype([("scale", "<f4"), ("zero_point", "<i4"), ("min_nudged", "<f4"), ("max_nudged", "<f4")])


class ConvDesc(Structure):
    _fields_ = [(n, c_int32) for n in ("batch", "h", "w", "c", "c_pitch_in", "n", "c_pitch_out", "kh", "kw",
                                       "stride", "pad", "wkind", "outkind")]


class Residual(Structure):
    _fields_ = [(n, c_int32) for n in ("t_zero_point", "t_act_min", "t_act_max", "t_mult", "s_zero_point", "s_mult", "rshift")]


class QtzError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what}: status {code} ({detail})")
        self.code = code


_lib = None

# name -> (restype, argtypes); every symbol declared in include/qtz.h
SIGNATURES = {
    "qtz_create": (c_int32, [POINTER(c_void_p), ctypes.c_int]),
    "qtz_destroy": (c_int32, [c_void_p]),
    "qtz_status_string": (c_char_p, [c_int32]),
    "qtz_last_error": (c_char_p, [c_void_p]),
    "qtz_last_device_status": (c_int32, [c_void_p, POINTER(c_int32), c_void_p]),
    "qtz_set_wait_budget": (c_int32, [c_void_p, c_int64]),
    "qtz_selftest_wait_timeout": (c_int32, [c_void_p, c_int64, c_void_p]),
    "qtz_probe_int8_peak": (c_int32, [c_void_p, c_int32, c_int32, POINTER(c_double), POINTER(c_float), c_void_p]),
    "qtz_probe_requant_rate": (c_int32, [c_void_p, c_int32, POINTER(c_double), POINTER(c_double), c_void_p]),
    "qtz_calibrate_minmax": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int32, c_void_p,
                                       c_void_p]),
    "qtz_minmax": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p]),
    "qtz_minmax_static": (c_int32, [c_void_p, c_int64, c_void_p, c_void_p]),
    "qtz_minmax_static_max_count": (c_int64, []),
    "qtz_range_state_bytes": (c_int64, [c_int64]),
    "qtz_range_reset": (c_int32, [c_void_p, c_void_p, c_int64, c_void_p]),
    "qtz_range_accumulate": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_double, c_void_p, c_void_p]),
    "qtz_range_finish": (c_int32, [c_void_p, c_void_p, c_int64, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                   POINTER(c_int32), c_void_p]),
    "qtz_params_from_range": (c_int32, [c_float, c_float, c_int32, c_int32, c_void_p]),
    "qtz_quantize_tensor": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_int32, c_int32,
                                      c_void_p, c_void_p]),
    "qtz_dequantize": (c_int32, [c_void_p, c_void_p, c_int32, c_int64, c_int64, c_int64, c_void_p, c_void_p,
                                 c_void_p]),
    "qtz_fold_batchnorm": (c_int32, [c_void_p] * 7 + [c_float, c_int64, c_int64, c_void_p, c_void_p, c_void_p]),
    "qtz_quantize_bias": (c_int32, [c_void_p, c_void_p, c_int64, c_float, c_void_p, c_int32, c_void_p, c_void_p]),
    "qtz_quantize_multiplier": (c_int32, [c_double, POINTER(c_int32), POINTER(c_int32)]),
    "qtz_activation_range": (c_int32, [c_int32, c_float, c_int32, POINTER(c_int32), POINTER(c_int32)]),
    "qtz_activation_range_bits": (c_int32, [c_int32, c_float, c_int32, c_int32, POINTER(c_int32), POINTER(c_int32)]),
    "qtz_pack_u4": (c_int32, [c_void_p, c_void_p, c_int64, c_int32, c_int32, c_void_p, c_int32, c_void_p]),
    "qtz_unpack_u4": (c_int32, [c_void_p, c_void_p, c_int64, c_int32, c_int32, c_void_p, c_int32, c_void_p]),
    "qtz_add_params": (c_int32, [c_float, c_float, c_float, POINTER(c_int32), POINTER(c_int32), POINTER(c_int32)]),
    "qtz_range_after_activation": (c_int32, [c_float, c_float, c_int32, POINTER(c_float), POINTER(c_float)]),
    "qtz_add_output_range": (c_int32, [c_void_p, c_void_p, c_int32, POINTER(c_float), POINTER(c_float)]),
    "qtz_accumulator_scales": (c_int32, [c_float, c_void_p, c_int64, c_void_p]),
    "qtz_requant_multipliers": (c_int32, [c_float, c_void_p, c_int64, c_float, c_void_p, c_void_p]),
    "qtz_avgpool_multiplier": (c_int32, [c_int32, c_float, c_float, POINTER(c_int32), POINTER(c_int32)]),
    "qtz_conv_create": (c_int32, [c_void_p, POINTER(ConvDesc), c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                  c_void_p, POINTER(c_void_p), c_void_p]),
    "qtz_conv_destroy": (c_int32, [c_void_p]),
    "qtz_conv_plan_kernel": (c_char_p, [c_void_p]),
    "qtz_conv_plan_detail": (c_char_p, [c_void_p]),
    "qtz_conv_set_profile_events": (c_int32, [c_void_p, c_void_p, c_void_p]),
    "qtz_conv2d_u8": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32, c_void_p]),
    "qtz_conv2d_add_u8": (c_int32, [c_void_p, c_void_p, c_int32, POINTER(Residual), c_void_p, c_void_p, c_int32, c_int32, c_int32,
                                    c_void_p]),
    "qtz_depthwise_u8": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32, c_void_p]),
    "qtz_conv2d_dw_pw_u8": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p, c_int32, c_int32,
                                      c_int32, c_void_p]),
    "qtz_add_u8": (c_int32, [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_int32, c_int32, c_int32, c_void_p,
                             c_int32, c_int32, c_int32, c_int64, c_int32, c_int32, c_void_p]),
    "qtz_simquant": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "qtz_sqnr": (c_int32, [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p]),
    "qtz_ema_update": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_double, POINTER(c_int32)]),
    "qtz_rescale_u8": (c_int32, [c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_int32, c_int32, c_int32, c_int64,
                                 c_int32, c_int32, c_int32, c_void_p]),
    "qtz_maxpool_u8": (c_int32, [c_void_p, c_void_p, c_void_p] + [c_int32] * 8 + [c_void_p]),
    "qtz_global_avgpool_u8": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p] + [c_int32] * 7 + [c_void_p]),
}


def load_library():
    """Opens libqtz.so and types its symbols.  Raises if the library has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1806_08342_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _np(a):
    return None if a is None else a.ctypes.data_as(c_void_p)


def _view(shape, axis):
    if axis is None:
        return 1, 1, int(np.prod(shape, dtype=np.int64))
    axis %= len(shape)
    return (int(np.prod(shape[:axis], dtype=np.int64)), int(shape[axis]),
            int(np.prod(shape[axis + 1:], dtype=np.int64)))


def _check_dev(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("expected contiguous CUDA tensors")


# ---- host-only helpers ------------------------------------------------------------------
def quantize_multiplier(real_multiplier):
    m, r = c_int32(), c_int32()
    rc = load_library().qtz_quantize_multiplier(float(real_multiplier), byref(m), byref(r))
    if rc:
        raise QtzError(rc, "qtz_quantize_multiplier")
    return m.value, r.value


def activation_range(kind, y_scale, y_zero_point):
    lo, hi = c_int32(), c_int32()
    rc = load_library().qtz_activation_range(kind, float(y_scale), int(y_zero_point), byref(lo), byref(hi))
    if rc:
        raise QtzError(rc, "qtz_activation_range")
    return lo.value, hi.value


def activation_range_bits(kind, y_scale, y_zero_point, bits):
    lo, hi = c_int32(), c_int32()
    rc = load_library().qtz_activation_range_bits(kind, float(y_scale), int(y_zero_point), int(bits), byref(lo), byref(hi))
    if rc:
        raise QtzError(rc, "qtz_activation_range_bits")
    return lo.value, hi.value


def add_params(a_scale, b_scale, y_scale):
    ma, mb, r = c_int32(), c_int32(), c_int32()
    rc = load_library().qtz_add_params(float(a_scale), float(b_scale), float(y_scale), byref(ma), byref(mb), byref(r))
    if rc:
        raise QtzError(rc, "qtz_add_params")
    return ma.value, mb.value, r.value


def range_after_activation(lo, hi, kind):
    a, b = c_float(), c_float()
    rc = load_library().qtz_range_after_activation(float(lo), float(hi), int(kind), byref(a), byref(b))
    if rc:
        raise QtzError(rc, "qtz_range_after_activation")
    return a.value, b.value


def add_output_range(a_params, b_params, kind):
    pa = np.ascontiguousarray(np.atleast_1d(a_params), dtype=QPARAMS)
    pb = np.ascontiguousarray(np.atleast_1d(b_params), dtype=QPARAMS)
    lo, hi = c_float(), c_float()
    rc = load_library().qtz_add_output_range(_np(pa), _np(pb), int(kind), byref(lo), byref(hi))
    if rc:
        raise QtzError(rc, "qtz_add_output_range")
    return lo.value, hi.value


def accumulator_scales(x_scale, w_params):
    wp = np.ascontiguousarray(np.atleast_1d(w_params), dtype=QPARAMS)
    out = np.zeros(wp.shape[0], QPARAMS)
    rc = load_library().qtz_accumulator_scales(float(x_scale), _np(wp), wp.shape[0], _np(out))
    if rc:
        raise QtzError(rc, "qtz_accumulator_scales")
    return out


def requant_multipliers(x_scale, w_params, y_scale):
    wp = np.ascontiguousarray(np.atleast_1d(w_params), dtype=QPARAMS)
    mult, rshift = np.zeros(wp.shape[0], np.int32), np.zeros(wp.shape[0], np.int32)
    rc = load_library().qtz_requant_multipliers(float(x_scale), _np(wp), wp.shape[0], float(y_scale), _np(mult), _np(rshift))
    if rc:
        raise QtzError(rc, "qtz_requant_multipliers")
    return mult, rshift


def avgpool_multiplier(hw, x_scale, y_scale):
    m, r = c_int32(), c_int32()
    rc = load_library().qtz_avgpool_multiplier(int(hw), float(x_scale), float(y_scale), byref(m), byref(r))
    if rc:
        raise QtzError(rc, "qtz_avgpool_multiplier")
    return m.value, r.value


def ema_update(state_lo, state_hi, batch_lo, batch_hi, decay, initialised):
    """Moving average of per-batch ranges (Section 2.5): updates the fp64 state arrays in place and
    returns the new `initialised` flag."""
    assert state_lo.dtype == np.float64 and state_hi.dtype == np.float64 and state_lo.shape == state_hi.shape
    batch_lo = np.ascontiguousarray(batch_lo, dtype=np.float32)
    batch_hi = np.ascontiguousarray(batch_hi, dtype=np.float32)
    assert batch_lo.size == state_lo.size and batch_hi.size == state_lo.size
    flag = c_int32(int(bool(initialised)))
    rc = load_library().qtz_ema_update(_np(state_lo), _np(state_hi), _np(batch_lo), _np(batch_hi), state_lo.size,
                                       float(decay), ctypes.byref(flag))
    if rc != 0:
        raise QtzError(rc, "qtz_ema_update")
    return bool(flag.value)


def params_from_range(lo, hi, bits=8, symmetric=False):
    q = np.zeros(1, QPARAMS)
    rc = load_library().qtz_params_from_range(float(lo), float(hi), bits, int(symmetric), _np(q))
    if rc:
        raise QtzError(rc, "qtz_params_from_range")
    return q[0]


def minmax_static(x, out=None):
    """qtz_minmax_static on the current device and stream.  `x`: fp32 CUDA tensor; returns a 3-word
    CUDA tensor (lo, hi, non-finite flag bits viewed as float).  Allocates only if `out` is None --
    pass a preallocated 3-element fp32 tensor to keep the call allocation-free."""
    _check_dev(x, out)
    assert x.dtype == torch.float32
    if out is None:
        out = torch.empty(3, dtype=torch.float32, device=x.device)
    rc = load_library().qtz_minmax_static(_ptr(x), x.numel(), _ptr(out), _stream())
    if rc:
        raise QtzError(rc, "qtz_minmax_static", load_library().qtz_status_string(rc).decode())
    return out


class Handle:
    """Owns a qtz_handle on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.h = c_void_p()
        self.device = device
        rc = self.lib.qtz_create(byref(self.h), device)
        if rc:
            raise QtzError(rc, "qtz_create", self.lib.qtz_status_string(rc).decode())

    def close(self):
        if self.h:
            self.lib.qtz_destroy(self.h)
            self.h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _chk(self, rc, what):
        if rc:
            detail = self.lib.qtz_status_string(rc).decode()
            if rc == -6:
                detail += ": " + self.lib.qtz_last_error(self.h).decode()
            raise QtzError(rc, what, detail)

    def device_status(self):
        site = c_int32()
        rc = self.lib.qtz_last_device_status(self.h, byref(site), _stream())
        return rc, site.value

    def set_wait_budget(self, cycles):
        self._chk(self.lib.qtz_set_wait_budget(self.h, int(cycles)), "qtz_set_wait_budget")

    def selftest_wait_timeout(self, budget_cycles):
        self._chk(self.lib.qtz_selftest_wait_timeout(self.h, int(budget_cycles), _stream()), "qtz_selftest_wait_timeout")

    def probe_int8_peak(self, mmas_per_cta=32768, launches=10):
        """(TOP/s, ms) of tcgen05.mma kind::i8 issued back to back on shared-memory resident operands."""
        tops, ms = c_double(), c_float()
        self._chk(self.lib.qtz_probe_int8_peak(self.h, int(mmas_per_cta), int(launches), byref(tops), byref(ms), _stream()),
                  "qtz_probe_int8_peak")
        return tops.value, ms.value

    def probe_requant_rate(self, kind):
        """(outputs per clock and SM at the maximum clock, outputs per second) of the requantising arithmetic."""
        a, b = c_double(), c_double()
        self._chk(self.lib.qtz_probe_requant_rate(self.h, int(kind), byref(a), byref(b), _stream()), "qtz_probe_requant_rate")
        return a.value, b.value

    def calibrate_minmax(self, x, axis=None, bits=8, symmetric=False):
        _check_dev(x)
        assert x.dtype == torch.float32
        o, a, i = _view(x.shape, axis)
        out = np.zeros(a, QPARAMS)
        self._chk(self.lib.qtz_calibrate_minmax(self.h, _ptr(x), o, a, i, bits, int(symmetric), _np(out),
                                                _stream()), "qtz_calibrate_minmax")
        return out

    def minmax(self, x, axis=None):
        _check_dev(x)
        assert x.dtype == torch.float32
        o, a, i = _view(x.shape, axis)
        lo, hi = np.zeros(a, np.float32), np.zeros(a, np.float32)
        self._chk(self.lib.qtz_minmax(self.h, _ptr(x), o, a, i, _np(lo), _np(hi), _stream()), "qtz_minmax")
        return lo, hi

    def range_state(self, axis_len=1):
        """A zeroed device buffer for range_accumulate (torch owns the memory)."""
        n = self.lib.qtz_range_state_bytes(int(axis_len))
        return torch.zeros(n // 8, dtype=torch.float64, device=f"cuda:{self.device}")

    def range_reset(self, state, axis_len=1):
        self._chk(self.lib.qtz_range_reset(self.h, _ptr(state), int(axis_len), _stream()), "qtz_range_reset")

    def range_accumulate(self, x, state, decay, axis=None):
        """Folds the min/max of batch `x` into the device-resident moving average; does not wait."""
        _check_dev(x, state)
        assert x.dtype == torch.float32
        o, a, i = _view(x.shape, axis)
        self._chk(self.lib.qtz_range_accumulate(self.h, _ptr(x), o, a, i, float(decay), _ptr(state), _stream()),
                  "qtz_range_accumulate")

    def range_finish(self, state, axis_len=1, bits=8, symmetric=False):
        """One blocking read: (lo, hi, params, batches) of the averaged ranges."""
        lo, hi = np.zeros(axis_len, np.float32), np.zeros(axis_len, np.float32)
        params = np.zeros(axis_len, QPARAMS)
        batches = c_int32()
        self._chk(self.lib.qtz_range_finish(self.h, _ptr(state), int(axis_len), bits, int(symmetric), _np(lo), _np(hi),
                                            _np(params), byref(batches), _stream()), "qtz_range_finish")
        return lo, hi, params, batches.value

    def quantize_tensor(self, x, params, axis=None, out_dtype=U8, restrict_range=False, out=None):
        _check_dev(x, out)
        assert x.dtype == torch.float32
        params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
        o, a, i = _view(x.shape, axis)
        assert params.shape[0] == a
        if out is None:
            if out_dtype in (S4_PACKED, U4_PACKED):
                run = i if i > 1 else a
                out = torch.empty((x.numel() // run) * ((run + 1) // 2), dtype=torch.uint8, device=x.device)
            else:
                out = torch.empty(x.shape, dtype={U8: torch.uint8, S8: torch.int8, U16: torch.uint16, S16: torch.int16}[out_dtype],
                                  device=x.device)
        self._chk(self.lib.qtz_quantize_tensor(self.h, _ptr(x), o, a, i, _np(params), out_dtype,
                                               int(restrict_range), _ptr(out), _stream()), "qtz_quantize_tensor")
        return out

    def dequantize(self, q, params, axis=None, in_dtype=None, shape=None, out=None):
        _check_dev(q, out)
        if in_dtype is None:
            in_dtype = {torch.uint8: U8, torch.int8: S8, torch.int32: S32, torch.uint16: U16,
                        torch.int16: S16}[q.dtype]                                    # packed 4-bit: pass in_dtype
        shape = tuple(q.shape) if shape is None else tuple(shape)
        params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
        o, a, i = _view(shape, axis)
        assert params.shape[0] == a
        if out is None:
            out = torch.empty(shape, dtype=torch.float32, device=q.device)
        self._chk(self.lib.qtz_dequantize(self.h, _ptr(q), in_dtype, o, a, i, _np(params), _ptr(out), _stream()),
                  "qtz_dequantize")
        return out

    def simquant(self, x, params, axis=None, code_dtype=U8, restrict_range=False, out=None):
        """SimQuant (Section 2.4): quantize then de-quantize, fp32 in and out."""
        _check_dev(x, out)
        assert x.dtype == torch.float32
        params = np.ascontiguousarray(np.atleast_1d(params), dtype=QPARAMS)
        o, a, i = _view(x.shape, axis)
        assert params.shape[0] == a
        if out is None:
            out = torch.empty_like(x)
        self._chk(self.lib.qtz_simquant(self.h, _ptr(x), o, a, i, _np(params), code_dtype, int(restrict_range),
                                        _ptr(out), _stream()), "qtz_simquant")
        return out

    def sqnr(self, w, w_hat, axis=None):
        """SQNR in dB (Appendix A) per index of `axis`, or of the whole tensor."""
        _check_dev(w, w_hat)
        assert w.dtype == torch.float32 and w_hat.dtype == torch.float32 and w.shape == w_hat.shape
        o, a, i = _view(w.shape, axis)
        out = np.zeros(a, np.float64)
        self._chk(self.lib.qtz_sqnr(self.h, _ptr(w), _ptr(w_hat), o, a, i, _np(out), _stream()), "qtz_sqnr")
        return out

    def rescale_u8(self, x, x_zp, mult, rshift, y_zp, act_min=0, act_max=255, c=None, out=None, out_offset=0):
        """uint8 tensor to another quantizer (concat, Section 3.2.1); with `out`, fills the channel
        slice [out_offset, out_offset + c) of that wider tensor."""
        _check_dev(x, out)
        xp = x.shape[-1]
        c = xp if c is None else c
        if out is None:
            out = torch.zeros_like(x)
        yp = out.shape[-1]
        dst = c_void_p(out.data_ptr() + out_offset)
        self._chk(self.lib.qtz_rescale_u8(self.h, _ptr(x), x_zp, mult, rshift, dst, y_zp, act_min, act_max,
                                          x.numel() // xp, c, xp, yp, _stream()), "qtz_rescale_u8")
        return out

    def pack_u4(self, x, c=None, out=None):
        """One 4-bit code per byte [..., pitch] -> two per byte [..., (c + 1) // 2 rounded up to 16]."""
        _check_dev(x, out)
        xp = x.shape[-1]
        c = xp if c is None else c
        if out is None:
            out = torch.zeros(x.shape[:-1] + (((c + 1) // 2 + 15) // 16 * 16,), dtype=torch.uint8, device=x.device)
        self._chk(self.lib.qtz_pack_u4(self.h, _ptr(x), x.numel() // xp, c, xp, _ptr(out), out.shape[-1], _stream()),
                  "qtz_pack_u4")
        return out

    def unpack_u4(self, x, c, out=None):
        _check_dev(x, out)
        xp = x.shape[-1]
        if out is None:
            out = torch.zeros(x.shape[:-1] + ((c + 15) // 16 * 16,), dtype=torch.uint8, device=x.device)
        self._chk(self.lib.qtz_unpack_u4(self.h, _ptr(x), x.numel() // xp, c, xp, _ptr(out), out.shape[-1], _stream()),
                  "qtz_unpack_u4")
        return out

    def fold_batchnorm(self, w, conv_bias, gamma, beta, mean, var, eps):
        _check_dev(w, conv_bias, gamma, beta, mean, var)
        n = w.shape[0]
        k = w.numel() // n
        w_inf = torch.empty_like(w)
        bias_inf = torch.empty(n, dtype=torch.float32, device=w.device)
        self._chk(self.lib.qtz_fold_batchnorm(self.h, _ptr(w), _ptr(conv_bias), _ptr(gamma), _ptr(beta), _ptr(mean),
                                              _ptr(var), float(eps), n, k, _ptr(w_inf), _ptr(bias_inf), _stream()),
                  "qtz_fold_batchnorm")
        return w_inf, bias_inf

    def quantize_bias(self, bias, x_scale, w_params, per_layer=False):
        _check_dev(bias)
        w_params = np.ascontiguousarray(np.atleast_1d(w_params), dtype=QPARAMS)
        n = bias.numel()
        out = torch.empty(n, dtype=torch.int32, device=bias.device)
        self._chk(self.lib.qtz_quantize_bias(self.h, _ptr(bias), n, float(x_scale), _np(w_params), int(per_layer),
                                             _ptr(out), _stream()), "qtz_quantize_bias")
        return out

    def conv_create(self, desc: ConvDesc, w_q, bias_q=None, w_zero_point=None, mult=None, rshift=None,
                    depthwise=False):
        _check_dev(w_q, bias_q)
        zw = None if w_zero_point is None else np.array([w_zero_point], np.int32)
        m = None if mult is None else np.ascontiguousarray(mult, dtype=np.int32)
        r = None if rshift is None else np.ascontiguousarray(rshift, dtype=np.int32)
        plan = c_void_p()
        self._chk(self.lib.qtz_conv_create(self.h, byref(desc), int(depthwise), _ptr(w_q), _ptr(bias_q), _np(zw),
                                           _np(m), _np(r), byref(plan), _stream()), "qtz_conv_create")
        return ConvPlan(self, plan, desc, depthwise)

    def add_u8(self, a, a_zp, a_mult, b, b_zp, b_mult, rshift, y_zp, act_min, act_max, c, out=None):
        _check_dev(a, b, out)
        pitch = a.shape[-1]
        pixels = a.numel() // pitch
        out = torch.empty_like(a) if out is None else out
        self._chk(self.lib.qtz_add_u8(self.h, _ptr(a), a_zp, a_mult, _ptr(b), b_zp, b_mult, rshift, _ptr(out), y_zp,
                                      act_min, act_max, pixels, c, pitch, _stream()), "qtz_add_u8")
        return out

    def maxpool_u8(self, x, c, k, stride, pad, out=None):
        _check_dev(x, out)
        b, hh, ww, pitch = x.shape
        oh, ow = (hh + 2 * pad - k) // stride + 1, (ww + 2 * pad - k) // stride + 1
        out = torch.empty((b, oh, ow, pitch), dtype=torch.uint8, device=x.device) if out is None else out
        self._chk(self.lib.qtz_maxpool_u8(self.h, _ptr(x), _ptr(out), b, hh, ww, c, pitch, k, stride, pad, _stream()),
                  "qtz_maxpool_u8")
        return out

    def global_avgpool_u8(self, x, x_zp, y_zp, mult, rshift, c, out=None):
        _check_dev(x, out)
        b, hh, ww, pitch = x.shape
        out = torch.empty((b, 1, 1, pitch), dtype=torch.uint8, device=x.device) if out is None else out
        self._chk(self.lib.qtz_global_avgpool_u8(self.h, _ptr(x), x_zp, _ptr(out), y_zp, mult, rshift, b, hh * ww, c,
                                                 pitch, _stream()), "qtz_global_avgpool_u8")
        return out


class ConvPlan:
    """Owns a qtz_conv_plan."""

    def __init__(self, handle: Handle, plan, desc: ConvDesc, depthwise: bool):
        self.handle, self.plan, self.desc, self.depthwise = handle, plan, desc, bool(depthwise)
        d = desc
        self.oh = (d.h + 2 * d.pad - d.kh) // d.stride + 1
        self.ow = (d.w + 2 * d.pad - d.kw) // d.stride + 1

    @property
    def kernel(self) -> str:
        return self.handle.lib.qtz_conv_plan_kernel(self.plan).decode()

    @property
    def detail(self) -> str:
        return self.handle.lib.qtz_conv_plan_detail(self.plan).decode()

    def empty_output(self, device):
        d = self.desc
        if d.outkind == OUT_S32_RAW:
            return torch.empty((d.batch, self.oh, self.ow, d.n), dtype=torch.int32, device=device)
        return torch.empty((d.batch, self.oh, self.ow, d.c_pitch_out), dtype=torch.uint8, device=device)

    def __call__(self, x, x_zero_point, y_zero_point=0, act_min=0, act_max=255, out=None):
        _check_dev(x, out)
        out = self.empty_output(x.device) if out is None else out
        fn = self.handle.lib.qtz_depthwise_u8 if self.depthwise else self.handle.lib.qtz_conv2d_u8
        self.handle._chk(fn(self.plan, _ptr(x), int(x_zero_point), _ptr(out), int(y_zero_point), int(act_min),
                            int(act_max), _stream()), "qtz_depthwise_u8" if self.depthwise else "qtz_conv2d_u8")
        return out

    def add_fused(self, x, x_zero_point, residual: Residual, s, y_zero_point, act_min, act_max, out=None):
        """qtz_conv2d_add_u8: this convolution and the element-wise add with `s` in one kernel."""
        _check_dev(x, s, out)
        out = self.empty_output(x.device) if out is None else out
        self.handle._chk(self.handle.lib.qtz_conv2d_add_u8(self.plan, _ptr(x), int(x_zero_point), byref(residual), _ptr(s),
                                                           _ptr(out), int(y_zero_point), int(act_min), int(act_max), _stream()),
                         "qtz_conv2d_add_u8")
        return out

    def after_depthwise(self, dw_plan, x, x_zero_point, mid_zero_point, mid_act_min, mid_act_max, y_zero_point, act_min,
                        act_max, out=None):
        """qtz_conv2d_dw_pw_u8: the 3x3 depthwise plan `dw_plan` and this pointwise plan in one kernel.  Raises
        QtzError (code ERR_UNSUPPORTED) when the pair cannot run fused."""
        _check_dev(x, out)
        out = self.empty_output(x.device) if out is None else out
        self.handle._chk(self.handle.lib.qtz_conv2d_dw_pw_u8(dw_plan.plan, self.plan, _ptr(x), int(x_zero_point),
                                                             int(mid_zero_point), int(mid_act_min), int(mid_act_max), _ptr(out),
                                                             int(y_zero_point), int(act_min), int(act_max), _stream()),
                         "qtz_conv2d_dw_pw_u8")
        return out

    def set_profile_events(self, start=None, stop=None):
        """start/stop: torch.cuda.Event(enable_timing=True) already created (recorded once), or None."""
        s = None if start is None else c_void_p(start.cuda_event)
        e = None if stop is None else c_void_p(stop.cuda_event)
        self.handle._chk(self.handle.lib.qtz_conv_set_profile_events(self.plan, s, e), "qtz_conv_set_profile_events")

    def close(self):
        if self.plan:
            self.handle.lib.qtz_conv_destroy(self.plan)
            self.plan = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def conv_desc(batch, h, w, c, n, kh, kw, stride, pad, wkind=W_S8_PER_CHANNEL_SYM, outkind=OUT_U8,
              c_pitch_in=None, c_pitch_out=None) -> ConvDesc:
    rup = lambda v: (v + 15) // 16 * 16
    return ConvDesc(batch, h, w, c, rup(c) if c_pitch_in is None else c_pitch_in, n,
                    rup(n) if c_pitch_out is None else c_pitch_out, kh, kw, stride, pad, wkind, outkind)
