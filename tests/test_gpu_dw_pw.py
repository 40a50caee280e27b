"""GPU parity of the fused depthwise -> pointwise block (qtz_conv2d_dw_pw_u8; Section 7: operator fusion) against the
oracle chain orc_depthwise_acc -> orc_requantize -> orc_conv2d_acc -> orc_requantize, bit for bit."""
import numpy as np
import pytest

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host, hq, pitched  # noqa: F401

pytestmark = pytest.mark.gpu


def multipliers(acc, gain):
    n = acc.shape[-1]
    span = np.abs(acc).reshape(-1, n).max(axis=0).astype(np.float64) + 1.0
    mr = [oracle.quantize_multiplier(float(v)) for v in gain / span]
    return np.array([m for m, _ in mr], np.int32), np.array([r for _, r in mr], np.int32)


def block_case(hq, b, h, w, c, n, stride, seed, z_x=None, mid=(0, 0, 255), out=(0, 0, 255)):
    g = synth.rng(seed, 90)
    x = pitched(synth.uniform_u8((b, h, w, c), seed, 2))
    z_x = int(g.integers(0, 256)) if z_x is None else z_x
    # depthwise layer (int8 per-channel symmetric weights), then its requantisation to the intermediate tensor
    wd = g.integers(-127, 128, size=(3, 3, c)).astype(np.int32)
    bd = g.integers(-3000, 3000, size=c).astype(np.int32)
    acc_d = oracle.depthwise_acc(x, z_x, wd, None, bd, stride, 1, c=c)
    md, rd = multipliers(acc_d, 150.0)
    assert rd.min() >= 32 and rd.max() <= 53
    z_m, lo_m, hi_m = mid
    t = oracle.requantize(acc_d, md, rd, z_m, lo_m, hi_m).astype(np.uint8)
    # pointwise layer on the intermediate tensor
    wp = g.integers(-127, 128, size=(n, 1, 1, c)).astype(np.int32)
    bp = g.integers(-20000, 20000, size=n).astype(np.int32)
    acc_p = oracle.conv2d_acc(t, z_m, wp, None, bp, 1, 0, c=c)
    mp, rp = multipliers(acc_p, 120.0)
    z_y, lo_y, hi_y = out
    want = oracle.requantize(acc_p, mp, rp, z_y, lo_y, hi_y)

    oh, ow = acc_d.shape[1:3]
    dw = hq.conv_create(qtz.conv_desc(b, h, w, c, c, 3, 3, stride, 1), dev(wd.astype(np.int8)), dev(bd), None, md, rd,
                        depthwise=True)
    pw = hq.conv_create(qtz.conv_desc(b, oh, ow, c, n, 1, 1, 1, 0), dev(wp.astype(np.int8)), dev(bp), None, mp, rp)
    xd = dev(x)
    fused = host(pw.after_depthwise(dw, xd, z_x, z_m, lo_m, hi_m, z_y, lo_y, hi_y))
    assert "depthwise-front" in pw.detail, pw.detail
    assert np.array_equal(fused[..., :n].astype(np.int32), want), pw.detail
    # and the same as the two kernels one after the other
    two = host(pw(dw(xd, z_x, z_m, lo_m, hi_m), z_m, z_y, lo_y, hi_y))
    assert np.array_equal(two[..., :n], fused[..., :n])
    return pw.detail


@pytest.mark.parametrize("b,h,w,c,n,stride", [
    (2, 16, 16, 32, 64, 1),        # one K block of 32 channels
    (2, 28, 28, 64, 128, 1),       # 64-byte K block
    (3, 14, 14, 128, 128, 1),      # 128-byte K block, whole images per tile
    (2, 28, 28, 256, 256, 1),      # two K blocks, full-width column tile
    (2, 30, 26, 128, 256, 2),      # stride 2, extents that no tile divides
    (2, 17, 19, 64, 32, 2),        # odd extents, stride 2, narrow output
    (1, 9, 9, 40, 24, 1),          # channels that fill neither a K block nor a 16-byte group
    (4, 7, 7, 256, 256, 1),        # tiles spanning several small images
    (5, 7, 7, 64, 96, 1),          # ... whose last tile runs past the batch
])
def test_block_shapes(hq, b, h, w, c, n, stride):
    block_case(hq, b, h, w, c, n, stride, seed=100 + c + n)


@pytest.mark.parametrize("z_x,mid,out", [
    (0, (0, 0, 255), (0, 0, 255)),            # between ReLU6 tensors: no padding refill, the saturating pack clamps
    (137, (12, 12, 200), (20, 20, 255)),      # padding cells refilled with z_x, explicit clamps on both layers
    (255, (255, 0, 255), (128, 0, 255)),      # extreme zero points
])
def test_block_zero_points_and_clamps(hq, z_x, mid, out):
    block_case(hq, 2, 20, 20, 128, 64, 1, seed=7, z_x=z_x, mid=mid, out=out)
    block_case(hq, 2, 21, 21, 64, 64, 2, seed=8, z_x=z_x, mid=mid, out=out)


def test_block_many_tiles_per_cta(hq):
    # more tiles than SMs: every CTA runs several, rings and accumulators wrap
    block_case(hq, 8, 56, 56, 128, 128, 1, seed=11)


def test_pairs_that_do_not_fuse_are_refused(hq):
    c = 64
    wd = dev(np.ones((3, 3, c), np.int8))
    ones = np.full(c, 1 << 30, np.int32)
    x = dev(np.zeros((1, 8, 8, c), np.uint8))
    dw = hq.conv_create(qtz.conv_desc(1, 8, 8, c, c, 3, 3, 1, 1), wd, None, None, ones, np.full(c, 40, np.int32), depthwise=True)
    # more than 256 output channels: several column tiles
    n = 512
    pw = hq.conv_create(qtz.conv_desc(1, 8, 8, c, n, 1, 1, 1, 0), dev(np.ones((n, 1, 1, c), np.int8)), None, None,
                        np.full(n, 1 << 30, np.int32), np.full(n, 40, np.int32))
    with pytest.raises(qtz.QtzError) as e:
        pw.after_depthwise(dw, x, 0, 0, 0, 255, 0, 0, 255)
    assert e.value.code == -3
    # a depthwise right shift below 32
    dw2 = hq.conv_create(qtz.conv_desc(1, 8, 8, c, c, 3, 3, 1, 1), wd, None, None, ones, np.full(c, 20, np.int32), depthwise=True)
    pw2 = hq.conv_create(qtz.conv_desc(1, 8, 8, c, 64, 1, 1, 1, 0), dev(np.ones((64, 1, 1, c), np.int8)), None, None,
                         np.full(64, 1 << 30, np.int32), np.full(64, 40, np.int32))
    with pytest.raises(qtz.QtzError) as e:
        pw2.after_depthwise(dw2, x, 0, 0, 0, 255, 0, 0, 255)
    assert e.value.code == -3
    # plans that do not chain
    pw3 = hq.conv_create(qtz.conv_desc(1, 8, 8, 32, 64, 1, 1, 1, 0), dev(np.ones((64, 1, 1, 32), np.int8)), None, None,
                         np.full(64, 1 << 30, np.int32), np.full(64, 40, np.int32))
    with pytest.raises(qtz.QtzError) as e:
        pw3.after_depthwise(dw, x, 0, 0, 0, 255, 0, 0, 255)
    assert e.value.code == -1
    # the refused calls launched nothing: the fusable pair still runs
    y = pw2.after_depthwise(dw, x, 0, 0, 0, 255, 0, 0, 255)
    assert host(y).shape[-1] >= 64
