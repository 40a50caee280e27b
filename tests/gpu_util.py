"""Helpers shared by the GPU parity tests (no arithmetic of the method lives here)."""
import numpy as np
import pytest
import torch


def rup16(v):
    return (v + 15) // 16 * 16


def pitched(x_np, pitch=None, fill=0xAB):
    """Copies [..., C] into [..., pitch] with a recognisable filler in the pad lanes."""
    c = x_np.shape[-1]
    pitch = rup16(c) if pitch is None else pitch
    out = np.full(x_np.shape[:-1] + (pitch,), fill, dtype=x_np.dtype)
    out[..., :c] = x_np
    return out


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


@pytest.fixture(scope="module")
def hq():
    from paper_1806_08342_b200 import qtz
    h = qtz.Handle(0)
    yield h
    rc, site = h.device_status()
    assert rc == 0, f"device status {rc} at site {site}"
    h.close()
