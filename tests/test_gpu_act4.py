"""4-bit activations (Section 3.2.4, Table 6) through the C ABI against the oracle: quantization to packed
4-bit codes, the storage round trip, convolution layers whose inputs AND outputs are 4-bit activations
(8-bit and 4-bit weights, dense and depthwise), and de-quantization of the packed result."""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq, pitched, rup16  # noqa: F401

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [(2, 7, 9, 24), (1, 5, 5, 17), (3, 16, 16, 64), (1, 1, 3, 1)])
def test_quantize_pack_unpack_dequantize_u4(hq, shape):
    x = synth.uniform_f32(shape, 71, shape[-1], -1.5, 4.0)
    c = shape[-1]
    xp_o = oracle.affine_params(x.min(), x.max(), 4)
    xp = hq.calibrate_minmax(dev(x), bits=4)
    assert xp[0].tobytes() == xp_o.tobytes()
    codes = oracle.quantize(x, xp_o, None, 0, 15).astype(np.uint8)
    packed = host(hq.quantize_tensor(dev(x), xp, axis=None, out_dtype=qtz.U4_PACKED))
    # the view is flat (axis None): nibbles run along the whole tensor
    want_flat = oracle.pack_u4(codes.reshape(1, -1))
    assert np.array_equal(packed.reshape(-1), want_flat.reshape(-1))
    back = host(hq.dequantize(dev(packed), xp, in_dtype=qtz.U4_PACKED, shape=shape))
    assert np.allclose(back, oracle.dequantize(codes, xp_o, None), rtol=1e-6, atol=0)
    # per-pixel storage: one code per byte <-> two per byte along the channels, pitched rows
    wide = pitched(codes, fill=0x0B)                                  # pad lanes hold a 4-bit value too
    p = host(hq.pack_u4(dev(wide), c))
    want = oracle.pack_u4(codes)
    assert np.array_equal(p[..., :(c + 1) // 2], want)
    u = host(hq.unpack_u4(dev(p), c))
    assert np.array_equal(u[..., :c], codes)
    # rows that are not 4-byte aligned take the generic path
    odd_pitch = np.zeros(shape[:-1] + (c + 3,), np.uint8)
    odd_pitch[..., :c] = codes
    p2 = torch.zeros(shape[:-1] + ((c + 1) // 2 + 1,), dtype=torch.uint8, device="cuda")
    hq.pack_u4(dev(odd_pitch), c, out=p2)
    assert np.array_equal(host(p2)[..., :(c + 1) // 2], want)


LAYERS = [  # batch, h, w, c, n, k, stride, depthwise, weight kind
    (2, 20, 20, 24, 40, 3, 1, False, qtz.W_S8_PER_CHANNEL_SYM),
    (3, 17, 13, 72, 136, 1, 1, False, qtz.W_S8_PER_CHANNEL_SYM),
    (2, 14, 14, 64, 32, 1, 1, False, qtz.W_S4_PACKED_PER_CHANNEL_SYM),
    (2, 15, 15, 48, 48, 3, 1, True, qtz.W_S8_PER_CHANNEL_SYM),
    (1, 30, 30, 3, 16, 3, 2, False, qtz.W_S8_PER_CHANNEL_SYM),
]


@pytest.mark.parametrize("layer", LAYERS)
def test_layer_with_four_bit_activations_in_and_out(hq, layer):
    b, h, w, c, n, k, stride, dw, wkind = layer
    pad = k // 2
    g = synth.rng(72, c * n)
    x = synth.uniform_f32((b, h, w, c), 72, c, 0.0, 6.0)
    wshape = (k, k, c) if dw else (n, k, k, c)
    wf = g.normal(0, 1.0 / np.sqrt(k * k * (1 if dw else c)), size=wshape).astype(np.float32)
    wbits = 4 if wkind == qtz.W_S4_PACKED_PER_CHANNEL_SYM else 8
    waxis = 2 if dw else 0
    # oracle side: 4-bit activation codes, per-channel weights, 4-bit output after ReLU6
    xp = oracle.affine_params(x.min(), x.max(), 4)
    xq = oracle.quantize(x, xp, None, 0, 15).astype(np.uint8)
    zx = int(xp["zero_point"])
    wp = oracle.calibrate_minmax(wf, waxis, wbits, True)
    wq = oracle.quantize(wf, wp, waxis, *oracle.code_range(wbits, 1, 1 if wbits == 8 else 0))
    acc = (oracle.depthwise_acc(xq, zx, wq, None, None, stride, pad) if dw
           else oracle.conv2d_acc(xq, zx, wq, None, None, stride, pad))
    ap = np.zeros(n, oracle.QPARAMS)
    ap["scale"] = np.float32(xp["scale"]) * wp["scale"]
    lo, hi = oracle.minmax(oracle.dequantize(acc, ap, 3))
    yp = oracle.affine_params(*oracle.range_after_activation(lo[0], hi[0], 2), 4)
    mr = [oracle.quantize_multiplier(float(xp["scale"]) * float(s) / float(yp["scale"])) for s in wp["scale"]]
    mult, rsh = np.array([m for m, _ in mr], np.int32), np.array([r for _, r in mr], np.int32)
    amin, amax = oracle.activation_range_bits(2, yp["scale"], int(yp["zero_point"]), 4)
    want = oracle.requantize(acc, mult, rsh, int(yp["zero_point"]), amin, amax).astype(np.uint8)
    assert want.max() <= 15 and len(np.unique(want)) >= 8

    # library side, from the packed activation tensor to the packed result
    g_xp = hq.calibrate_minmax(dev(x), bits=4)
    assert g_xp[0].tobytes() == xp.tobytes()
    flat = hq.quantize_tensor(dev(x), g_xp, out_dtype=qtz.U4_PACKED)          # nibbles along the flat tensor
    if c % 2 == 0:                                                             # then a pixel's channels fill whole bytes
        assert np.array_equal(host(flat).reshape(b, h, w, c // 2), oracle.pack_u4(xq))
    x_packed = dev(np.ascontiguousarray(pitched(oracle.pack_u4(xq), fill=0)))
    x_codes = hq.unpack_u4(x_packed, c)
    assert np.array_equal(host(x_codes)[..., :c], xq)
    if wkind == qtz.W_S4_PACKED_PER_CHANNEL_SYM:
        api_w = oracle.pack_s4(wq.reshape(n, -1))
    else:
        api_w = wq.astype(np.int8)
    assert qtz.activation_range_bits(2, yp["scale"], int(yp["zero_point"]), 4) == (amin, amax)
    desc = qtz.conv_desc(b, h, w, c, n, k, k, stride, pad, wkind)
    plan = hq.conv_create(desc, dev(api_w), None, None, mult, rsh, depthwise=dw)
    y = plan(x_codes, zx, int(yp["zero_point"]), amin, amax)
    assert np.array_equal(host(y)[..., :n], want)
    y_packed = hq.pack_u4(y, n)
    assert np.array_equal(host(y_packed)[..., :(n + 1) // 2], oracle.pack_u4(want))
    # dequantized 4-bit outputs agree with the oracle's within 1e-6 relative
    tight = np.ascontiguousarray(host(y_packed)[..., :(n + 1) // 2]) if n % 2 == 0 else None
    if tight is not None:
        real = host(hq.dequantize(dev(tight), yp, in_dtype=qtz.U4_PACKED, shape=want.shape))
        assert np.allclose(real, oracle.dequantize(want.astype(np.int32), yp, None), rtol=1e-6, atol=0)
