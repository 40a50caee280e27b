"""GPU parity of qtz_conv2d_u8 / qtz_depthwise_u8 against the oracle: every uint8 / int32
output bit-exact.  Shapes span several tiles with ragged tails, the degenerate cases, every
weight kind, and the first two workloads (single 3x3 conv; quantized GEMM)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq, pitched, rup16  # noqa: F401

pytestmark = pytest.mark.gpu


def make_weights(wkind, shape, seed):
    """Random weight codes in the API layout plus the oracle's int32 view and zero point."""
    g = synth.rng(seed, 70)
    if wkind == qtz.W_S8_PER_CHANNEL_SYM:
        codes = g.integers(-127, 128, size=shape).astype(np.int32)
        codes.flat[0] = -128                                       # raw codes may use the full range
        return codes.astype(np.int8), codes, None
    if wkind == qtz.W_U8_PER_LAYER_ASYM:
        codes = g.integers(0, 256, size=shape).astype(np.int32)
        return codes.astype(np.uint8), codes, int(g.integers(64, 192))
    codes = g.integers(-8, 8, size=shape).astype(np.int32)
    codes.flat[0] = -8
    return None, codes, None                                        # packed by the caller (layout differs)


def conv_case(hq, b, h, w, c, n, k, stride, pad, wkind, seed, raw=False, act=0, expect_kernel=None, real_m=None, bias_range=20000,
              expect_detail=None, in_pitch=None):
    x = synth.uniform_u8((b, h, w, c), seed, 1)
    xp = pitched(x, in_pitch)
    api_w, codes, zw = make_weights(wkind, (n, k, k, c), seed)
    if wkind == qtz.W_S4_PACKED_PER_CHANNEL_SYM:
        api_w = oracle.pack_s4(codes.reshape(n, -1))
    g = synth.rng(seed, 71)
    bias = g.integers(-bias_range, bias_range, size=n).astype(np.int32)
    z_x = int(g.integers(64, 192))
    z_w = None if zw is None else np.full(n, zw, np.int32)
    acc = oracle.conv2d_acc(xp, z_x, codes, z_w, bias, stride, pad, c=c)
    desc = qtz.conv_desc(b, h, w, c, n, k, k, stride, pad, wkind, qtz.OUT_S32_RAW if raw else qtz.OUT_U8, c_pitch_in=in_pitch)
    if raw:
        plan = hq.conv_create(desc, dev(api_w), dev(bias), zw)
        got = host(plan(dev(xp), z_x))
        if expect_kernel:
            assert plan.kernel == expect_kernel
        if expect_detail:
            assert expect_detail in plan.detail, plan.detail
        assert got.shape == acc.shape
        assert np.array_equal(got, acc)
        return
    # per-channel multipliers spread over two decades so that outputs use the whole code range
    span = np.abs(acc).reshape(-1, n).max(axis=0).astype(np.float64) + 1.0
    if real_m is None:
        real_m = 100.0 / span * np.exp(g.uniform(-1.0, 1.0, size=n))
    mr = [oracle.quantize_multiplier(float(v)) for v in real_m]
    mult = np.array([m for m, _ in mr], np.int32)
    rsh = np.array([r for _, r in mr], np.int32)
    z_y = int(g.integers(100, 156))
    lo, hi = {0: (0, 255), 1: (z_y, 255), 2: (z_y, min(255, z_y + 120))}[act]
    want = oracle.requantize(acc, mult, rsh, z_y, lo, hi)
    plan = hq.conv_create(desc, dev(api_w), dev(bias), zw, mult, rsh)
    if expect_kernel:
        assert plan.kernel == expect_kernel
    got = host(plan(dev(xp), z_x, z_y, lo, hi))
    if expect_detail:
        assert expect_detail in plan.detail, plan.detail
    assert got.shape[:3] == want.shape[:3]
    bad = np.argwhere(got[..., :n].astype(np.int32) != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[0]}: got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"
    assert want.size < 2000 or len(np.unique(want)) > 20             # the case is not degenerate


# 4-bit weights stay packed in global memory and are expanded to int8 in shared memory (Section 7: compressed
# weight storage decompressed on the fly) whenever a CTA's column tile of the layer fits on chip
INT4_SMEM_SHAPES = [
    # b, h, w, c, n, k, stride, pad, raw
    (2, 28, 28, 96, 24, 1, 1, 0, False),      # pointwise, 64-byte... K block of 128 with a ragged tail
    (3, 20, 20, 32, 64, 3, 1, 1, False),      # 3x3 with border classes
    (1, 40, 40, 40, 200, 1, 1, 0, False),     # K block of 64, wide output
    (2, 30, 30, 16, 8, 1, 1, 0, False),       # K block of 32
    (256, 1, 1, 1792, 1000, 1, 1, 0, True),   # a classifier: several column tiles, one tile per CTA, raw logits
    (2, 64, 64, 3, 48, 3, 2, 1, False),       # an image stem (row-window form)
    (1, 12, 12, 144, 24, 1, 2, 0, False),     # strided pointwise
]


@pytest.mark.parametrize("shape", INT4_SMEM_SHAPES)
def test_int4_weights_expanded_in_shared_memory(hq, shape):
    b, h, w, c, n, k, stride, pad, raw = shape
    conv_case(hq, b, h, w, c, n, k, stride, pad, qtz.W_S4_PACKED_PER_CHANNEL_SYM, 900 + c + n, raw=raw,
              expect_kernel="tcgen05", expect_detail="int4-expanded-in-smem")


def test_int4_weights_too_large_for_shared_memory_are_streamed(hq):
    conv_case(hq, 4, 28, 28, 448, 1792, 1, 1, 0, qtz.W_S4_PACKED_PER_CHANNEL_SYM, 950, expect_kernel="tcgen05",
              expect_detail="weights:streamed")


STEM_SHAPES = [
    # b, h, w, c, n, k, stride, pad
    (2, 17, 15, 3, 32, 3, 2, 1),      # MobileNet stem shape (3 input channels, stride 2)
    (1, 23, 21, 3, 64, 7, 2, 3),      # ResNet stem shape
    (1, 20, 250, 3, 256, 7, 2, 3),    # stems whose weights do not stay resident (they share ring stages with the frame
    (1, 12, 14, 4, 272, 5, 2, 2),     # runs), several tiles per output row (125 columns), two column tiles
    (2, 11, 260, 3, 32, 3, 2, 1),     # several output rows per tile, two tiles per output row, a ragged last row group
    (1, 10, 12, 5, 32, 5, 1, 2),      # a stride-1 stem (16-byte frame pixels), four output rows per tile
    (1, 9, 9, 5, 7, 3, 1, 1),         # odd channel counts, n not a multiple of 4
    (3, 6, 7, 20, 70, 1, 1, 0),       # pointwise, ragged n tile
    (1, 8, 8, 16, 16, 3, 1, 0),       # no padding
    (1, 5, 5, 300, 10, 3, 1, 1),      # K = 2700 spans several K chunks
    (1, 1, 1, 8, 8, 1, 1, 0),         # single output pixel
    (1, 9, 9, 160, 24, 3, 2, 1),      # strided 3x3 with a long reduction (K = 1440): the CUDA-core fallback
    (2, 11, 9, 130, 20, 5, 1, 2),     # 5x5 with K = 3250: fallback as well
]


@pytest.mark.parametrize("shape", STEM_SHAPES)
@pytest.mark.parametrize("wkind", [qtz.W_S8_PER_CHANNEL_SYM, qtz.W_U8_PER_LAYER_ASYM,
                                   qtz.W_S4_PACKED_PER_CHANNEL_SYM])
def test_conv_generic_shapes(hq, shape, wkind):
    long_k = shape[5] * shape[5] * shape[3] > 1024 and shape[5] > 1 and not (shape[5] == 3 and shape[6] == 1 and shape[7] == 1)
    conv_case(hq, *shape, wkind, seed=100 + shape[1], expect_kernel="direct" if long_k else "tcgen05")


@pytest.mark.parametrize("shape", STEM_SHAPES[:4])
def test_conv_raw_int32_output(hq, shape):
    conv_case(hq, *shape, qtz.W_U8_PER_LAYER_ASYM, seed=7, raw=True)
    conv_case(hq, *shape, qtz.W_S8_PER_CHANNEL_SYM, seed=8, raw=True)


@pytest.mark.parametrize("act", [0, 1, 2])
def test_conv_activation_clamps(hq, act):
    conv_case(hq, 1, 12, 12, 16, 24, 3, 1, 1, qtz.W_S8_PER_CHANNEL_SYM, seed=20 + act, act=act)


# ---- layers the tensor-core path is meant for (1x1 / GEMM / 3x3 stride 1 pad 1) ------------
TC_SHAPES = [
    (1, 32, 32, 16, 32, 3, 1, 1),     # the single-conv workload's geometry (M=1024, K=144, N=32)
    (2, 14, 14, 64, 96, 3, 1, 1),     # small image: pixel tiles span images
    (3, 7, 7, 128, 48, 3, 1, 1),      # 7x7 image, C a full 128-byte K block
    (1, 20, 18, 24, 40, 3, 1, 1),     # C = 24 (pitch 32), ragged tiles both ways
    (4, 10, 10, 32, 64, 1, 1, 0),     # pointwise, M = 400: three full tiles and a ragged one
    (1, 33, 31, 88, 136, 1, 1, 0),    # MobileNet-v2-1.4 widths, nothing a multiple of 16
    (1, 16, 16, 256, 272, 1, 1, 0),   # two K blocks, N beyond one 256 tile
    (2, 9, 9, 512, 24, 1, 1, 0),      # long K, narrow N
    (1, 12, 12, 64, 32, 1, 2, 0),     # strided pointwise (ResNet down-sampling shortcut)
    (3, 15, 13, 256, 512, 1, 2, 0),   # ... odd extents, several images, two K blocks, two column tiles
    (2, 56, 56, 40, 72, 1, 3, 0),     # ... stride 3, many pixel tiles
    (2, 24, 24, 32, 128, 1, 1, 0),    # pointwise outputs of 128, 192, 256 and 8 channels: whole tiles leave as one
    (1, 40, 40, 48, 192, 1, 1, 0),    # contiguous run (rows of 8, 12, 16 and 1 sixteen-byte pieces, staged in
    (1, 30, 30, 64, 256, 1, 1, 0),    # rotated order), several tiles and a short last one
    (1, 50, 50, 16, 8, 1, 1, 0),
]


@pytest.mark.parametrize("shape", TC_SHAPES)
@pytest.mark.parametrize("wkind", [qtz.W_S8_PER_CHANNEL_SYM, qtz.W_U8_PER_LAYER_ASYM,
                                   qtz.W_S4_PACKED_PER_CHANNEL_SYM])
def test_conv_tensor_core_shapes(hq, shape, wkind):
    conv_case(hq, *shape, wkind, seed=200 + shape[3], expect_kernel="tcgen05")


@pytest.mark.parametrize("shape", TC_SHAPES[:5])
def test_conv_tensor_core_raw(hq, shape):
    conv_case(hq, *shape, qtz.W_U8_PER_LAYER_ASYM, seed=300 + shape[3], raw=True, expect_kernel="tcgen05")


@pytest.mark.parametrize("lo_m,hi_m", [(0.26, 0.49), (0.13, 0.49), (0.26, 0.99), (0.3, 3.0)])
def test_conv_large_multipliers(hq, lo_m, hi_m):
    # Real multipliers near 1 (4-bit weights make them large): right shifts of 32 (still the folded
    # fast form), mixed 32/33+, 31 and below (the general 64-bit form).  One input channel keeps the
    # accumulators small enough for the outputs to spread over the code range.
    n = 40
    real_m = np.exp(np.linspace(np.log(lo_m), np.log(hi_m), n))
    shifts = {oracle.quantize_multiplier(float(v))[1] for v in real_m}
    assert (min(shifts) <= 32) and (hi_m < 0.5 or min(shifts) <= 31)
    conv_case(hq, 3, 20, 20, 1, n, 1, 1, 0, qtz.W_S4_PACKED_PER_CHANNEL_SYM, seed=401, real_m=real_m, expect_kernel="tcgen05", bias_range=60)
    conv_case(hq, 2, 13, 13, 2, n, 3, 1, 1, qtz.W_S8_PER_CHANNEL_SYM, seed=402, real_m=real_m / 40.0 if hi_m > 1 else real_m / 64.0, bias_range=2000)


def test_extreme_zero_points_and_codes(hq):
    # all-255 inputs against all -128 / 255 weights with zero points at both ends
    for wkind, wval, zw in [(qtz.W_S8_PER_CHANNEL_SYM, -128, None), (qtz.W_U8_PER_LAYER_ASYM, 255, 0),
                            (qtz.W_U8_PER_LAYER_ASYM, 0, 255)]:
        b, h, w, c, n = 1, 6, 6, 64, 16
        x = np.full((b, h, w, c), 255, np.uint8)
        codes = np.full((n, 3, 3, c), wval, np.int32)
        api_w = codes.astype(np.int8 if wkind == qtz.W_S8_PER_CHANNEL_SYM else np.uint8)
        for z_x in (0, 255):
            z_w = None if zw is None else np.full(n, zw, np.int32)
            acc = oracle.conv2d_acc(x, z_x, codes, z_w, None, 1, 1)
            desc = qtz.conv_desc(b, h, w, c, n, 3, 3, 1, 1, wkind, qtz.OUT_S32_RAW)
            plan = hq.conv_create(desc, dev(api_w), None, zw)
            assert np.array_equal(host(plan(dev(x), z_x)), acc)


# ---- workload 1: one quantized 3x3 convolution, every API call once -------------------------
def test_single_conv_workload_end_to_end(hq):
    t = synth.single_conv(seed=1)
    x, w, bias = t["x"], t["w"], t["bias"]
    n = w.shape[0]
    # oracle side
    xq_p = oracle.calibrate_minmax(x)
    wq_p = oracle.calibrate_minmax(w, 0, 8, True)
    xq = oracle.quantize(x, xq_p, None, 0, 255).astype(np.uint8)
    wq = oracle.quantize(w, wq_p, 0, -127, 127)
    bq = oracle.quantize_bias(bias, xq_p["scale"][0], wq_p["scale"])
    z_x = int(xq_p["zero_point"][0])
    acc = oracle.conv2d_acc(xq, z_x, wq, None, bq, 1, 1)
    acc_p = np.zeros(n, oracle.QPARAMS)
    acc_p["scale"] = (xq_p["scale"][0].astype(np.float32) * wq_p["scale"]).astype(np.float32)
    real = np.clip(oracle.dequantize(acc, acc_p, 3), 0.0, 6.0)       # ReLU6 on the real values
    yq_p = oracle.calibrate_minmax(real)
    mr = [oracle.quantize_multiplier(float(xq_p["scale"][0]) * float(s) / float(yq_p["scale"][0]))
          for s in wq_p["scale"]]
    mult, rsh = [m for m, _ in mr], [r for _, r in mr]
    z_y = int(yq_p["zero_point"][0])
    lo, hi = oracle.activation_range(2, yq_p["scale"][0], z_y)
    want = oracle.requantize(acc, np.array(mult, np.int32), np.array(rsh, np.int32), z_y, lo, hi)

    # GPU side: the same steps through the C ABI
    xd, wd = dev(x), dev(w)
    g_xp = hq.calibrate_minmax(xd)
    g_wp = hq.calibrate_minmax(wd, axis=0, symmetric=True)
    assert g_xp.tobytes() == xq_p.tobytes() and g_wp.tobytes() == wq_p.tobytes()
    assert z_x == 0 and np.isclose(float(g_xp["scale"][0]), 6.0 / 255.0, rtol=1e-3)
    g_xq = hq.quantize_tensor(xd, g_xp)
    g_wq = hq.quantize_tensor(wd, g_wp, axis=0, out_dtype=qtz.S8, restrict_range=True)
    g_bq = hq.quantize_bias(dev(bias), g_xp["scale"][0], g_wp)
    assert np.array_equal(host(g_xq), xq) and np.array_equal(host(g_wq).astype(np.int32), wq)
    assert np.array_equal(host(g_bq), bq)
    raw_plan = hq.conv_create(qtz.conv_desc(1, 32, 32, 16, n, 3, 3, 1, 1, outkind=qtz.OUT_S32_RAW), g_wq, g_bq)
    g_acc = raw_plan(g_xq, z_x)
    assert np.array_equal(host(g_acc), acc)
    g_lo, g_hi = hq.minmax(hq.dequantize(g_acc, acc_p, axis=3))       # ReLU6 clamps the range itself
    g_yp = np.atleast_1d(qtz.params_from_range(min(max(g_lo[0], 0.0), 6.0), min(max(g_hi[0], 0.0), 6.0)))
    assert g_yp.tobytes() == yq_p.tobytes()
    g_mr = [qtz.quantize_multiplier(float(g_xp["scale"][0]) * float(s) / float(g_yp["scale"][0]))
            for s in g_wp["scale"]]
    assert [m for m, _ in g_mr] == mult and [r for _, r in g_mr] == rsh
    assert qtz.activation_range(2, g_yp["scale"][0], z_y) == (lo, hi)
    plan = hq.conv_create(qtz.conv_desc(1, 32, 32, 16, n, 3, 3, 1, 1), g_wq, g_bq, None, mult, rsh)
    got = host(plan(g_xq, z_x, z_y, lo, hi))
    assert np.array_equal(got[..., :n].astype(np.int32), want)
    # dequantized output agrees with the oracle's within 1e-6 relative
    g_out = host(hq.dequantize(dev(np.ascontiguousarray(got[..., :n])), g_yp))
    o_out = oracle.dequantize(want, yq_p, None)
    assert np.allclose(g_out, o_out, rtol=1e-6, atol=0)


# ---- workload 2: quantized GEMM, both operands asymmetric uint8 ------------------------------
def gemm_case(hq, m, n, k, seed=2, rows=None):
    t = synth.gemm_u8(m, n, k, seed)
    a, b = t["a"], t["b"]
    bt = np.ascontiguousarray(b.T).reshape(n, 1, 1, k)                # OHWI view of B
    rows = np.arange(m) if rows is None else rows
    ap = pitched(a)
    acc = oracle.conv2d_acc(a[rows].reshape(len(rows), 1, 1, k), t["z_a"], bt.astype(np.int32),
                            np.full(n, t["z_b"], np.int32), t["bias"], 1, 0).reshape(len(rows), n)
    # one per-layer output quantizer from the accumulator range, replicated per channel
    span = float(np.abs(acc).max()) + 1.0
    m_q, r_q = oracle.quantize_multiplier(127.0 / span)
    mult, rsh = np.full(n, m_q, np.int32), np.full(n, r_q, np.int32)
    z_y = 128
    want = oracle.requantize(acc, mult, rsh, z_y, 0, 255)
    desc = qtz.conv_desc(m, 1, 1, k, n, 1, 1, 1, 0, qtz.W_U8_PER_LAYER_ASYM)
    plan = hq.conv_create(desc, dev(bt), dev(t["bias"]), t["z_b"], mult, rsh)
    got = host(plan(dev(ap.reshape(m, 1, 1, -1)), t["z_a"], z_y, 0, 255)).reshape(m, -1)
    assert np.array_equal(got[rows][:, :n].astype(np.int32), want)
    assert len(np.unique(want)) > 50
    assert plan.kernel == "tcgen05"
    # GEMM-like layers (full-width column tiles, long reduction, at least a tile per SM) run on CTA pairs
    assert ("cta-pairs" in plan.detail) == (n >= 2048 and k >= 2048 and (m // 128) * (n // 256) >= 296), plan.detail
    return plan.kernel


@pytest.mark.parametrize("size", [512, 1024, 2048, 4096, 8192])
def test_gemm_workload_full_parity(hq, size):
    # every row of every size: each 128-row pixel tile, each band of the tile rasterisation and each column
    # tile is compared element by element (the oracle needs about half a minute for the three large sizes)
    gemm_case(hq, size, size, size)


def test_gemm_ragged(hq):
    gemm_case(hq, 300, 200, 136)
    gemm_case(hq, 129, 17, 1000)


# ---- depthwise ---------------------------------------------------------------------------------
DW_SHAPES = [(2, 14, 14, 32, 1), (1, 15, 13, 64, 2), (3, 7, 7, 24, 1), (1, 9, 10, 136, 2),
             (2, 5, 5, 1024, 1), (1, 1, 1, 16, 1), (1, 2, 3, 8, 2), (1, 112, 112, 32, 1)]


@pytest.mark.parametrize("shape", DW_SHAPES)
@pytest.mark.parametrize("wkind", [qtz.W_S8_PER_CHANNEL_SYM, qtz.W_U8_PER_LAYER_ASYM,
                                   qtz.W_S4_PACKED_PER_CHANNEL_SYM])
def test_depthwise(hq, shape, wkind):
    depthwise_case(hq, shape, wkind, 150.0)


@pytest.mark.parametrize("gain", [4000.0, 30000.0])
def test_depthwise_large_multipliers(hq, gain):
    # multipliers around 0.3 (right shift 32, still the fast form) and above 1 (general form)
    depthwise_case(hq, (2, 12, 12, 40, 1), qtz.W_S4_PACKED_PER_CHANNEL_SYM, gain)


def depthwise_case(hq, shape, wkind, gain):
    b, h, w, c, stride = shape
    x = pitched(synth.uniform_u8((b, h, w, c), 31, c))
    api_w, codes, zw = make_weights(wkind, (3, 3, c), 31 + c)
    if wkind == qtz.W_S4_PACKED_PER_CHANNEL_SYM:
        api_w = oracle.pack_s4(codes.reshape(9, c))
    g = synth.rng(31, 72)
    bias = g.integers(-3000, 3000, size=c).astype(np.int32)
    z_x = int(g.integers(0, 256))
    z_w = None if zw is None else np.full(c, zw, np.int32)
    acc = oracle.depthwise_acc(x, z_x, codes, z_w, bias, stride, 1, c=c)
    span = np.abs(acc).reshape(-1, c).max(axis=0).astype(np.float64) + 1.0
    mr = [oracle.quantize_multiplier(float(v)) for v in gain / span]
    mult = np.array([m for m, _ in mr], np.int32)
    rsh = np.array([r for _, r in mr], np.int32)
    if gain > 1000.0:
        assert rsh.min() <= 32
    z_y = 30
    want = oracle.requantize(acc, mult, rsh, z_y, z_y, 255)
    desc = qtz.conv_desc(b, h, w, c, c, 3, 3, stride, 1, wkind)
    plan = hq.conv_create(desc, dev(api_w), dev(bias), zw, mult, rsh, depthwise=True)
    assert plan.kernel == "depthwise"
    got = host(plan(dev(x), z_x, z_y, z_y, 255))
    assert np.array_equal(got[..., :c].astype(np.int32), want)


def test_conv_argument_errors(hq):
    w = dev(np.zeros((8, 3, 3, 16), np.int8))
    ones = np.full(8, 1 << 30, np.int32), np.full(8, 31, np.int32)
    with pytest.raises(qtz.QtzError) as e:                                       # K too long
        hq.conv_create(qtz.conv_desc(1, 8, 8, 4096, 8, 3, 3, 1, 1), w, None, None, *ones)
    assert e.value.code == -4
    with pytest.raises(qtz.QtzError) as e:                                       # bad pitch
        hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 8, 3, 3, 1, 1, c_pitch_in=24), w, None, None, *ones)
    assert e.value.code == -2
    with pytest.raises(qtz.QtzError) as e:                                       # missing z_w
        hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 8, 3, 3, 1, 1, qtz.W_U8_PER_LAYER_ASYM), w, None, None, *ones)
    assert e.value.code == -1
    with pytest.raises(qtz.QtzError) as e:                                       # 5x5 depthwise
        hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 16, 5, 5, 1, 2), w, None, None, np.ones(16, np.int32),
                       np.ones(16, np.int32), depthwise=True)
    assert e.value.code == -3
    plan = hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 8, 3, 3, 1, 1), w, None, None, *ones)
    x = dev(np.zeros((1, 8, 8, 16), np.uint8))
    y = plan.empty_output(x.device)
    lib = hq.lib
    assert lib.qtz_conv2d_u8(plan.plan, x.data_ptr(), 256, y.data_ptr(), 0, 0, 255, None) == -1
    assert lib.qtz_conv2d_u8(plan.plan, x.data_ptr(), 0, y.data_ptr(), 0, 10, 5, None) == -1
    assert lib.qtz_conv2d_u8(plan.plan, x.data_ptr() + 4, 0, y.data_ptr(), 0, 0, 255, None) == -2
    assert lib.qtz_depthwise_u8(plan.plan, x.data_ptr(), 0, y.data_ptr(), 0, 0, 255, None) == -1


# ---- convolution with the residual add fused into its epilogue (Section 3.2.1, Section 7) ---------------------
FUSED_ADD_SHAPES = [
    # b, h, w, c, n, k, weight kind, add scales (t, s, y)
    (3, 20, 20, 64, 256, 1, qtz.W_S8_PER_CHANNEL_SYM, (0.02, 0.03, 0.04)),          # ResNet projection back to 4x width
    (2, 14, 14, 32, 64, 3, qtz.W_S8_PER_CHANNEL_SYM, (0.05, 0.01, 0.05)),           # 3x3 tiles (4-D boxes, border classes)
    (2, 28, 28, 144, 24, 1, qtz.W_S4_PACKED_PER_CHANNEL_SYM, (0.03, 0.03, 0.045)),   # MobileNet-v2 linear bottleneck, ragged box
    (1, 9, 9, 256, 1000, 1, qtz.W_S8_PER_CHANNEL_SYM, (0.02, 0.02, 0.03)),          # several column tiles
    (2, 12, 12, 48, 136, 1, qtz.W_U8_PER_LAYER_ASYM, (1e-3, 2e-3, 900.0)),          # add shift above 38: 64-bit form
    (2, 12, 12, 48, 40, 1, qtz.W_S8_PER_CHANNEL_SYM, (40.0, 25.0, 0.0005)),         # add shift 10..15: funnel-shift form
    (1, 10, 10, 32, 32, 1, qtz.W_S8_PER_CHANNEL_SYM, (4000.0, 100.0, 0.0005)),      # add shift below 10: 64-bit shift
]


@pytest.mark.parametrize("shape", FUSED_ADD_SHAPES)
@pytest.mark.parametrize("alias", [False, True])
def test_conv_with_fused_residual_add(hq, shape, alias):
    b, h, w, c, n, k, wkind, (st, ss, sy) = shape
    pad = k // 2
    seed = 1200 + n
    x = pitched(synth.uniform_u8((b, h, w, c), seed, 1))
    api_w, codes, zw = make_weights(wkind, (n, k, k, c), seed)
    if wkind == qtz.W_S4_PACKED_PER_CHANNEL_SYM:
        api_w = oracle.pack_s4(codes.reshape(n, -1))
    g = synth.rng(seed, 71)
    bias = g.integers(-20000, 20000, size=n).astype(np.int32)
    z_x, z_t, z_s, z_y = (int(v) for v in g.integers(60, 190, size=4))
    z_w = None if zw is None else np.full(n, zw, np.int32)
    acc = oracle.conv2d_acc(x, z_x, codes, z_w, bias, 1, pad, c=c)
    span = np.abs(acc).reshape(-1, n).max(axis=0).astype(np.float64) + 1.0
    mr = [oracle.quantize_multiplier(float(v)) for v in 100.0 / span * np.exp(g.uniform(-1.0, 1.0, size=n))]
    mult, rsh = np.array([m for m, _ in mr], np.int32), np.array([r for _, r in mr], np.int32)
    t_lo, t_hi = 0, 255                                   # a linear layer before the add
    t = oracle.requantize(acc, mult, rsh, z_t, t_lo, t_hi).astype(np.uint8)
    s = pitched(synth.uniform_u8((b, h, w, n), seed, 2), fill=0)
    m_t, m_s, r = oracle.add_params(np.float32(st), np.float32(ss), np.float32(sy))
    lo, hi = z_y, 255                                     # ReLU after the add
    want = oracle.add_u8(t, z_t, m_t, s[..., :n], z_s, m_s, r, z_y, lo, hi)
    assert {0.04: 16 <= r <= 38, 900.0: r >= 39, 0.0005: r < 16}.get(sy, True)
    if 0.01 < sy < 1.0:
        assert len(np.unique(want)) > 20
    desc = qtz.conv_desc(b, h, w, c, n, k, k, 1, pad, wkind)
    plan = hq.conv_create(desc, dev(api_w), dev(bias), zw, mult, rsh)
    res = qtz.Residual(z_t, t_lo, t_hi, m_t, z_s, m_s, r)
    s_dev = dev(s)
    y = plan.add_fused(dev(x), z_x, res, s_dev, z_y, lo, hi, out=s_dev if alias else None)
    assert "+residual-add" in plan.detail
    assert np.array_equal(host(y)[..., :n], want)
    # and it is what the two separate calls give
    t_dev = plan(dev(x), z_x, z_t, t_lo, t_hi)
    assert np.array_equal(host(t_dev)[..., :n], t)
    two = hq.add_u8(t_dev, z_t, m_t, dev(s), z_s, m_s, r, z_y, lo, hi, n)
    assert np.array_equal(host(two)[..., :n], want)


def test_fused_residual_add_is_refused_where_it_cannot_run(hq):
    w = dev(synth.uniform_s8((3, 3, 16), 1300, 0))
    m, r = oracle.quantize_multiplier(0.01)
    dw = hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 16, 3, 3, 1, 1), w, None, None, np.full(16, m, np.int32),
                        np.full(16, r, np.int32), depthwise=True)
    x = dev(np.zeros((1, 8, 8, 16), np.uint8))
    with pytest.raises(qtz.QtzError) as e:
        dw.add_fused(x, 0, qtz.Residual(0, 0, 255, 1 << 30, 0, 1 << 30, 31), x, 0, 0, 255)
    assert e.value.code == -1
    raw = hq.conv_create(qtz.conv_desc(1, 8, 8, 16, 16, 1, 1, 1, 0, outkind=qtz.OUT_S32_RAW),
                         dev(synth.uniform_s8((16, 1, 1, 16), 1300, 1)), None)
    with pytest.raises(qtz.QtzError) as e:
        raw.add_fused(x, 0, qtz.Residual(0, 0, 255, 1 << 30, 0, 1 << 30, 31), x, 0, 0, 255,
                      out=torch.zeros((1, 8, 8, 16), dtype=torch.int32, device="cuda"))
    assert e.value.code == -3


@pytest.mark.parametrize("shape", [(16, 14, 14, 256, 512), (16, 7, 7, 512, 2048), (17, 14, 14, 256, 512), (5, 9, 9, 64, 1000)])
def test_few_pixel_tiles_spread_over_column_tiles(hq, shape):
    # a layer with few pixel tiles is split into narrow column tiles so that it covers the SMs; the split must not
    # leave a role waiting for a column tile that lies beyond the real channels (the status word would say so)
    b, h, w, c, n = shape
    conv_case(hq, b, h, w, c, n, 1, 1, 0, qtz.W_S8_PER_CHANNEL_SYM, 1400 + n, expect_kernel="tcgen05")
    torch.cuda.synchronize()
    assert hq.device_status() == (0, 0)


# ---- requantisation forms the workloads rarely reach ---------------------------------------------------------
@pytest.mark.parametrize("k,c,n", [(1, 32, 48), (3, 16, 32)])
def test_requant_right_shifts_above_53(hq, k, c, n):
    # real multipliers near 2e-8 give right shifts of 56 (the general 64-bit form); with int32 biases near +-1.9e9
    # the outputs still spread over the code range
    g = synth.rng(1500 + k, 0)
    real_m = 2e-8 * np.exp(g.uniform(-0.6, 0.6, size=n))
    assert all(54 <= oracle.quantize_multiplier(float(v))[1] <= 62 for v in real_m)
    conv_case(hq, 2, 12, 12, c, n, k, 1, k // 2, qtz.W_S8_PER_CHANNEL_SYM, 1500 + k, real_m=real_m, bias_range=1_900_000_000)
    torch.cuda.synchronize()
    assert hq.device_status() == (0, 0)


@pytest.mark.parametrize("k,c,n", [(1, 64, 40), (3, 32, 40)])
def test_requant_large_values_with_small_shifts(hq, k, c, n):
    # multipliers of 1..2 (right shift 30) and biases near 1e9: a requantised value can leave 32 bits before the
    # clamp, so the narrow forms are not allowed and the 64-bit form must be taken
    g = synth.rng(1510 + k, 0)
    real_m = np.exp(g.uniform(0.05, 0.6, size=n))
    assert all(oracle.quantize_multiplier(float(v))[1] == 30 for v in real_m)
    conv_case(hq, 1, 6, 6, c, n, k, 1, k // 2, qtz.W_S8_PER_CHANNEL_SYM, 1510 + k, real_m=real_m, bias_range=1_000_000_000)
    # the same multipliers with accumulators small enough for the narrow form (shift below 32, values within 32 bits)
    conv_case(hq, 1, 6, 6, c, n, k, 1, k // 2, qtz.W_S8_PER_CHANNEL_SYM, 1520 + k, real_m=real_m / 4000.0, bias_range=2000)


def test_layer_whose_accumulator_can_leave_int32_is_refused(hq):
    # K 255 max|w| + |bias| beyond int32: the oracle reports overflow for the worst input, the library refuses the layer
    c, n = 64, 16
    w = np.full((n, 1, 1, c), 127, np.int8)
    bias = np.full(n, 2_147_000_000, np.int32)
    x = np.full((1, 2, 2, c), 255, np.uint8)
    with pytest.raises(oracle.OracleError) as e:
        oracle.conv2d_acc(x, 0, w.astype(np.int32), None, bias, 1, 0)
    assert e.value.code == -4
    m, r = oracle.quantize_multiplier(1e-6)
    with pytest.raises(qtz.QtzError) as e:
        hq.conv_create(qtz.conv_desc(1, 2, 2, c, n, 1, 1, 1, 0), dev(w), dev(bias), None, np.full(n, m, np.int32), np.full(n, r, np.int32))
    assert e.value.code == -4
    with pytest.raises(qtz.QtzError) as e:
        hq.conv_create(qtz.conv_desc(1, 2, 2, c, n, 1, 1, 1, 0, outkind=qtz.OUT_S32_RAW), dev(w), dev(bias))
    assert e.value.code == -4
    ok = hq.conv_create(qtz.conv_desc(1, 2, 2, c, n, 1, 1, 1, 0, outkind=qtz.OUT_S32_RAW), dev(w), dev(bias // 2))
    assert np.array_equal(host(ok(dev(x), 0)), oracle.conv2d_acc(x, 0, w.astype(np.int32), None, bias // 2, 1, 0))


def test_back_to_back_layers_on_ping_pong_buffers(hq):
    """Kernels of consecutive layers are launched as programmatic dependents: a layer's prologue may run while the
    layer before it is still finishing, but no activation may be read, and no output written, before that layer is
    done.  Four layers alternate between two buffers (each layer's output overwrites the input of the layer before
    it) and are enqueued back to back several times; every result must be the oracle's."""
    b, h, w, c = 32, 40, 40, 64
    g = synth.rng(1700, 0)
    x0 = synth.uniform_u8((b, h, w, c), 1700, 1)
    m, r = oracle.quantize_multiplier(1.0 / 900.0)
    mult, rsh = np.full(c, m, np.int32), np.full(c, r, np.int32)
    md, rd = oracle.quantize_multiplier(1.0 / 120.0)
    multd, rshd = np.full(c, md, np.int32), np.full(c, rd, np.int32)
    layers, want, cur = [], [], x0
    for i in range(4):
        if i % 2 == 0:
            wq = g.integers(-127, 128, size=(c, 1, 1, c)).astype(np.int8)
            plan = hq.conv_create(qtz.conv_desc(b, h, w, c, c, 1, 1, 1, 0), dev(wq), None, None, mult, rsh)
            acc = oracle.conv2d_acc(cur, 0, wq.astype(np.int32), None, None, 1, 0)
            cur = oracle.requantize(acc, mult, rsh, 0, 0, 255).astype(np.uint8)
        else:
            wq = g.integers(-127, 128, size=(3, 3, c)).astype(np.int8)
            plan = hq.conv_create(qtz.conv_desc(b, h, w, c, c, 3, 3, 1, 1), dev(wq), None, None, multd, rshd, depthwise=True)
            acc = oracle.depthwise_acc(cur, 0, wq.astype(np.int32), None, None, 1, 1)
            cur = oracle.requantize(acc, multd, rshd, 0, 0, 255).astype(np.uint8)
        layers.append(plan)
        want.append(cur)
    assert len(np.unique(want[-1])) > 30
    bufs = [torch.empty((b, h, w, c), dtype=torch.uint8, device="cuda") for _ in range(2)]
    x_dev = dev(x0)
    for rep in range(5):
        bufs[0].copy_(x_dev)
        outs = []
        for i, plan in enumerate(layers):                     # buffer 0 -> 1 -> 0 -> 1 -> 0, nothing in between
            plan(bufs[i % 2], 0, 0, 0, 255, out=bufs[(i + 1) % 2])
        torch.cuda.synchronize()
        assert np.array_equal(host(bufs[0]), want[3]), rep      # the last layer wrote buffer 0
        # and every intermediate, one layer at a time
        bufs[0].copy_(x_dev)
        for i, plan in enumerate(layers):
            plan(bufs[i % 2], 0, 0, 0, 255, out=bufs[(i + 1) % 2])
            assert np.array_equal(host(bufs[(i + 1) % 2]), want[i]), (rep, i)
    assert hq.device_status() == (0, 0)


@pytest.mark.parametrize("case", [
    # b, h, w, c, n, k, stride, weight kind, input pitch, expected form
    (2, 64, 64, 3, 32, 3, 2, qtz.W_S8_PER_CHANNEL_SYM, 4, "row-window"),      # MobileNet stem, images at 4 bytes per pixel
    (2, 60, 60, 3, 64, 7, 2, qtz.W_S8_PER_CHANNEL_SYM, 4, "row-window"),      # ResNet stem
    (1, 33, 31, 3, 48, 3, 2, qtz.W_S4_PACKED_PER_CHANNEL_SYM, 4, "row-window"),
    (2, 30, 30, 6, 24, 3, 2, qtz.W_S8_PER_CHANNEL_SYM, 8, "row-window"),      # 8-byte pixels
    (2, 30, 30, 3, 24, 3, 2, qtz.W_U8_PER_LAYER_ASYM, 4, "im2col"),           # asymmetric weights: explicit im2col
    (1, 20, 20, 4, 16, 5, 1, qtz.W_S8_PER_CHANNEL_SYM, 4, "row-window"),      # stride 1: 16-byte frame pixels
])
def test_image_stems_take_narrow_pixel_pitches(hq, case):
    b, h, w, c, n, k, stride, wkind, pitch, form = case
    conv_case(hq, b, h, w, c, n, k, stride, k // 2, wkind, 1800 + c + n + k, expect_kernel="tcgen05", expect_detail=form, in_pitch=pitch)
    conv_case(hq, b, h, w, c, n, k, stride, k // 2, wkind, 1900 + c + n + k, raw=True, in_pitch=pitch)


def test_narrow_pixel_pitch_is_refused_elsewhere(hq):
    m, r = oracle.quantize_multiplier(0.01)
    for args, dw in [((1, 8, 8, 4, 16, 1, 1, 1, 0), False), ((1, 8, 8, 8, 8, 3, 3, 1, 1), True)]:
        w = dev(synth.uniform_s8((3, 3, 8) if dw else (16, 1, 1, 4), 1990, 0))
        n = args[4]
        with pytest.raises(qtz.QtzError) as e:
            hq.conv_create(qtz.conv_desc(*args, c_pitch_in=args[3]), w, None, None, np.full(n, m, np.int32), np.full(n, r, np.int32), depthwise=dw)
        assert e.value.code == -2
