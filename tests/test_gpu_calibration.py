"""Streaming activation calibration on the GPU (Section 2.5: moving average of per-batch min/max over
many batches, Section 3.1.2) against the oracle's three steps: orc_minmax of every batch,
orc_ema_update of the fp64 state, orc_affine_params of the state rounded to fp32.  The device keeps
the running state; the host reads it once at the end."""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import hq  # noqa: F401

pytestmark = pytest.mark.gpu


def batches(n, shape, seed):
    # activations whose range drifts from batch to batch, as it does over a calibration set
    return [synth.normal_f32(shape, seed, 10 + i, std=1.0 + 0.3 * i, mean=0.5 - 0.1 * i) for i in range(n)]


@pytest.mark.parametrize("axis,shape", [(None, (4, 19, 23, 24)), (3, (3, 9, 11, 40)), (None, (1, 1, 1, 5)),
                                        (None, (2, 150, 150, 33))])
@pytest.mark.parametrize("decay", [0.9, 0.0, 0.99])
def test_moving_average_of_ranges_over_batches(hq, axis, shape, decay):
    xs = batches(7, shape, 300)
    n = 1 if axis is None else shape[axis]
    state = hq.range_state(n)
    o_lo, o_hi, o_init = np.zeros(n), np.zeros(n), False
    for x in xs:
        hq.range_accumulate(torch.from_numpy(x).cuda(), state, decay, axis=axis)      # enqueued, never waited on
        blo, bhi = oracle.minmax(x, axis)
        o_init = oracle.ema_update(o_lo, o_hi, blo, bhi, decay, o_init)
    lo, hi, params, count = hq.range_finish(state, n)
    assert count == len(xs)
    assert np.array_equal(lo.view(np.uint32), o_lo.astype(np.float32).view(np.uint32))
    assert np.array_equal(hi.view(np.uint32), o_hi.astype(np.float32).view(np.uint32))
    for i in range(n):
        want = oracle.affine_params(np.float32(o_lo[i]), np.float32(o_hi[i]), 8)
        assert params[i].tobytes() == want.tobytes(), (i, params[i], want)
    # the state itself holds the fp64 averages bit for bit (header of 16 bytes, then lo[n], hi[n])
    raw = state.cpu().numpy()
    assert np.array_equal(raw[2:2 + n].view(np.uint64), o_lo.view(np.uint64))
    assert np.array_equal(raw[2 + n:2 + 2 * n].view(np.uint64), o_hi.view(np.uint64))


def test_streaming_calibration_feeds_a_quantizer_and_rejects_bad_batches(hq):
    xs = batches(5, (2, 30, 30, 16), 301)
    state = hq.range_state(1)
    with pytest.raises(qtz.QtzError) as e:                      # nothing accumulated yet
        hq.range_finish(state, 1)
    assert e.value.code == -1
    for x in xs[:3]:
        hq.range_accumulate(torch.from_numpy(x).cuda(), state, 0.9)
    _, _, good, _ = hq.range_finish(state, 1)
    bad = xs[3].copy()
    bad[1, 7, 7, 3] = np.inf
    hq.range_accumulate(torch.from_numpy(bad).cuda(), state, 0.9)
    with pytest.raises(qtz.QtzError) as e:
        hq.range_finish(state, 1)
    assert e.value.code == -5
    raw = state.cpu().numpy()
    assert raw[:1].view(np.int32)[0] == 3                       # the bad batch was not folded in
    # the parameters drive the quantizer exactly as the oracle's would
    x = xs[4]
    want = oracle.quantize(x, good, None, 0, 255).astype(np.uint8)
    got = hq.quantize_tensor(torch.from_numpy(x).cuda(), good).cpu().numpy()
    assert np.array_equal(got, want)
    # a reset starts a new average; symmetric 4-bit parameters from the same state
    hq.range_reset(state, 1)
    hq.range_accumulate(torch.from_numpy(xs[0]).cuda(), state, 0.5)
    lo, hi, params, count = hq.range_finish(state, 1, bits=4, symmetric=True)
    blo, bhi = oracle.minmax(xs[0])
    assert count == 1 and lo[0] == blo[0] and hi[0] == bhi[0]
    assert params[0].tobytes() == oracle.symmetric_params(blo[0], bhi[0], 4).tobytes()
    for args in [(1.0,), (-0.1,)]:
        with pytest.raises(qtz.QtzError):
            hq.range_accumulate(torch.from_numpy(xs[0]).cuda(), state, *args)
