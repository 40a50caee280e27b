"""qtz_minmax_static: the range reduction for callers that may not allocate device memory
(a server whose own pool already owns the whole GPU, or a loop that cannot take the device-wide
synchronisation an allocation may cause).  Its partial results live in a fixed array inside the
library instead of a cudaMalloc'ed buffer, so the check that matters is that it returns exactly
what the allocating entry point qtz_minmax returns -- also on a second call, which finds the
previous call's partials still sitting in the shared array.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  It must pass alone in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_08342_b200 import qtz, synth

pytestmark = pytest.mark.gpu


def test_static_minmax_matches_allocating_entry_point_twice_in_a_row():
    hq = qtz.Handle(0)
    out = torch.empty(3, dtype=torch.float32, device="cuda")           # the caller's output buffer
    # first call: many blocks' worth of partials; second call: fewer blocks and other values, so
    # stale partials of the first call would change the answer if they were ever read
    first = torch.from_numpy(synth.normal_f32((3 * 65536 + 1234,), 41, 1, std=5.0, mean=1.0)).cuda()
    second = torch.from_numpy(synth.uniform_f32((65536 + 77,), 41, 2, -0.25, 0.5)).cuda()
    for x in (first, second):
        want_lo, want_hi = hq.minmax(x)
        got = qtz.minmax_static(x, out=out)
        torch.cuda.synchronize()
        g = got.cpu().numpy()
        assert g[0] == want_lo[0] and g[1] == want_hi[0]               # min/max are exact: same bits
        assert g[2:].view(np.uint32)[0] == 0
        o_lo, o_hi = oracle.minmax(x.cpu().numpy())                     # and what the oracle's definition gives
        assert g[0] == o_lo[0] and g[1] == o_hi[0]
    # misaligned start and a NaN: same verdicts as the allocating call
    got = qtz.minmax_static(first[3:1000], out=out).cpu().numpy()
    lo, hi = hq.minmax(first[3:1000])
    assert got[0] == lo[0] and got[1] == hi[0]
    bad = second.clone()
    bad[65600] = float("nan")                                          # lands in the second block
    assert qtz.minmax_static(bad, out=out).cpu().numpy()[2:].view(np.uint32)[0] != 0
    with pytest.raises(qtz.QtzError):
        hq.minmax(bad)
    hq.close()


def test_static_minmax_rejects_sizes_beyond_its_fixed_capacity():
    lib = qtz.load_library()
    cap = lib.qtz_minmax_static_max_count()
    assert cap == 1 << 28
    x = torch.zeros(16, dtype=torch.float32, device="cuda")
    out = torch.empty(3, dtype=torch.float32, device="cuda")
    rc = lib.qtz_minmax_static(x.data_ptr(), cap + 1, out.data_ptr(), None)   # refused before any launch
    assert rc == -9 and b"capacity" in lib.qtz_status_string(rc)
    assert lib.qtz_minmax_static(None, 16, out.data_ptr(), None) == -1
    assert lib.qtz_minmax_static(x.data_ptr(), 0, out.data_ptr(), None) == -1


def test_static_minmax_chunk_boundaries_and_no_allocation():
    """One partial covers 65 536 values: sizes on either side of that boundary, a 16-byte aligned start with
    a tail that is not a multiple of four, and the promise itself -- after the first call on the device (which
    loads the kernels and looks the array's address up) a call leaves the amount of free device memory as it was."""
    out = torch.empty(3, dtype=torch.float32, device="cuda")
    base = synth.normal_f32((2 * 65536 + 64,), 43, 1, std=3.0)
    dev_x = torch.from_numpy(base).cuda()
    qtz.minmax_static(dev_x[:16], out=out)                              # the per-device set-up happens here
    torch.cuda.synchronize()
    for count in (1, 3, 65535, 65536, 65537, 2 * 65536 - 1, 2 * 65536 + 1, 65536 + 7):
        free_before = torch.cuda.mem_get_info()[0]
        g = qtz.minmax_static(dev_x[:count], out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, count       # nothing was allocated or freed
        lo, hi = oracle.minmax(base[:count])
        g = g.cpu().numpy()
        assert g[0] == lo[0] and g[1] == hi[0] and g[2:].view(np.uint32)[0] == 0, count
