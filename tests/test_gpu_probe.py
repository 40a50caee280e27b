"""The bounded-wait path and the tensor-core probe, through the C ABI.

Every mbarrier wait of the convolution kernels carries a cycle budget; when it runs out the kernel
records a status word and returns.  Here that path runs for real, in its harmless form: a single CTA
waits on a barrier nothing signals and must come back by itself (no trap, no fault, no hang), after
which the handle reports the timeout and its site, and the context is as usable as before.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth
from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def small_conv(hq):
    x = synth.uniform_u8((2, 9, 9, 32), 90, 0)
    w = synth.uniform_s8((16, 1, 1, 32), 90, 1)
    m, r = oracle.quantize_multiplier(1.0 / 900.0)
    mult, rsh = np.full(16, m, np.int32), np.full(16, r, np.int32)
    plan = hq.conv_create(qtz.conv_desc(2, 9, 9, 32, 16, 1, 1, 1, 0), dev(w), None, None, mult, rsh)
    got = host(plan(dev(x), 5, 100, 0, 255))[..., :16]
    want = oracle.requantize(oracle.conv2d_acc(x, 5, w.astype(np.int32), None, None, 1, 0), mult, rsh, 100, 0, 255)
    assert np.array_equal(got.astype(np.int32), want)
    plan.close()


def test_wait_that_nothing_signals_gives_up_and_reports():
    hq = qtz.Handle(0)
    assert hq.device_status() == (0, 0)
    hq.selftest_wait_timeout(20000)                     # about ten microseconds of SM clocks
    torch.cuda.synchronize()                            # the kernel came back by itself
    rc, site = hq.device_status()
    assert (rc, site) == (-7, 8)
    assert hq.device_status() == (0, 0)                 # reading the status clears it
    small_conv(hq)                                      # the context is still good
    assert hq.device_status() == (0, 0)
    # the budget of the convolution kernels is settable; a sane budget changes no result
    hq.set_wait_budget(50_000_000)
    small_conv(hq)
    assert hq.device_status() == (0, 0)
    for bad in (0, 999):
        with pytest.raises(qtz.QtzError):
            hq.set_wait_budget(bad)
    with pytest.raises(qtz.QtzError):
        hq.selftest_wait_timeout(0)
    hq.close()


def test_int8_tensor_core_probe_reports_a_plausible_rate():
    hq = qtz.Handle(0)
    tops, ms = hq.probe_int8_peak(mmas_per_cta=4096, launches=5)
    assert hq.device_status() == (0, 0)
    # dense int8 on this part is nominally 4.5 POP/s; anything between a fifth of that and a little above it is a
    # measurement, anything else means the loop did not do the work it counts
    assert 900.0 < tops < 5200.0, (tops, ms)
    hq.close()


def test_requant_rate_probe_orders_its_three_kinds():
    hq = qtz.Handle(0)
    taps, _ = hq.probe_requant_rate(0)
    requant, _ = hq.probe_requant_rate(1)
    both, per_s = hq.probe_requant_rate(2)
    # taps and requantisation share one pipe: together they are slower than either, and no faster than their
    # harmonic sum by more than the loop overhead they share
    assert both < min(taps, requant) and both > 0.8 / (1.0 / taps + 1.0 / requant), (taps, requant, both)
    assert 4.0 < both < 20.0 and per_s > 1e12
    hq.close()
