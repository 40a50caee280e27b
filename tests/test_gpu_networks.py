"""GPU parity of whole-network integer inference (the MobileNet-v1, ResNet-50 and MobileNet-v2-1.4
workloads) against the oracle: every activation tensor of every layer and the int32 logits must be
bit-exact, and every derived quantizer must be the same record.

Small-batch cases compare all images at full 224x224 resolution; the full-batch cases (128 / 256
images, the launch configuration the benchmark uses) compare the calibration images plus sampled
images, which the oracle computes one by one (images are independent once the quantizers are fixed).
"""
import hashlib
import json
import os

import numpy as np
import pytest
import torch

from oracle import netrun
from paper_1806_08342_b200 import network, qtz, synth
from gpu_util import hq  # noqa: F401

pytestmark = pytest.mark.gpu

CASES = {"mobilenet_v1": 8, "resnet50": 8, "mobilenet_v2_14": 4}   # network -> weight bits


def compare(net, got, want, rows=None, skip=()):
    checked = 0
    for name, w in want.items():
        if name in skip:
            continue
        g = got[name].cpu().numpy()
        if rows is not None:
            g = g[rows]
        if name == "logits":
            assert np.array_equal(g, w["q"]), name
            continue
        c = w["q"].shape[-1]
        bad = np.argwhere(g[..., :c] != w["q"])
        assert bad.size == 0, f"{name}: {len(bad)} mismatches, first {bad[0]}"
        if name != "in":
            assert net.params[name].tobytes() == w["p"].tobytes(), name
        checked += 1
    return checked


@pytest.mark.parametrize("name", list(CASES))
def test_network_small_batch_every_layer(hq, name):
    ops = synth.NETWORKS[name]()
    images = synth.network_input(3, 224, 11)
    want = netrun.run(ops, images, 2, 11, CASES[name])
    net = network.QuantizedNetwork(hq, ops, 11, CASES[name])
    got = net.build(images, 2)
    torch.cuda.synchronize()
    assert compare(net, got, want) >= len([o for o in ops if o["op"] != "fc"])
    # the timed pass (plans reused, outputs overwritten) reproduces the same tensors
    for t in got.values():
        if t.dtype == torch.uint8 and t is not got["in"]:
            t.zero_()
    net.forward()
    torch.cuda.synchronize()
    # (a convolution fused with the residual add after it never stores its own output)
    compare(net, got, want, skip=net.fused_away)
    if name != "mobilenet_v1":
        assert len(net.fused_away) >= 10 and any(k[0] == "conv+add" for k in net.schedule)
    logits = want["logits"]["q"]
    assert len(np.unique(logits)) > 500                              # not a degenerate network
    kinds = {L.plan.kernel for L in net.layers if L.op["op"] in ("conv", "fc")}
    assert "tcgen05" in kinds                                         # stems included (explicit im2col)


def test_network_with_fused_depthwise_blocks(hq):
    """MobileNet-v1 with every depthwise -> pointwise pair the library can fuse run as one kernel: the tensors the
    timed pass still writes equal the oracle's, the intermediate tensors are never stored."""
    ops = synth.NETWORKS["mobilenet_v1"]()
    images = synth.network_input(3, 224, 11)
    want = netrun.run(ops, images, 2, 11, 8)
    net = network.QuantizedNetwork(hq, ops, 11, 8, fuse_depthwise=True)
    got = net.build(images, 2)
    torch.cuda.synchronize()
    blocks = [item for item in net.schedule if item[0] == "dw+pw"]
    assert len(blocks) >= 5, [item[0] for item in net.schedule]
    assert all("depthwise-front" in item[1].plan.detail for item in blocks)
    for key, t in got.items():
        if t.dtype == torch.uint8 and key != "in":
            t.zero_()
    net.forward()
    torch.cuda.synchronize()
    assert all(not got[key].any() for key in net.fused_away)          # never written by the timed pass
    compare(net, got, want, skip=net.fused_away)
    rc, site = hq.device_status()
    assert rc == 0, (rc, site)


@pytest.mark.parametrize("name,batch", [("mobilenet_v1", 128), ("resnet50", 256), ("mobilenet_v2_14", 256)])
def test_network_full_batch_sampled_images(hq, name, batch):
    ops = synth.NETWORKS[name]()
    images = synth.network_input(batch, 224, 12)
    rows = np.array([0, 1, batch // 2 + 3, batch - 1])
    want = netrun.run(ops, images[rows], 2, 12, CASES[name])          # calibration images first
    net = network.QuantizedNetwork(hq, ops, 12, CASES[name])
    got = net.build(images, 2)
    torch.cuda.synchronize()
    compare(net, got, want, rows)
    rc, site = hq.device_status()
    assert rc == 0, (rc, site)


GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "network_hashes.json")


@pytest.mark.parametrize("name", list(CASES))
def test_network_full_batch_every_image(hq, name):
    """The whole batch the benchmark runs (128 / 256 images), every tensor of every layer: the SHA-256 of the
    library's codes and quantizer record must equal the digest the oracle alone wrote
    (tests/golden/make_network_hashes.py, which imports nothing of the CUDA library)."""
    table = json.load(open(GOLDEN))
    if name not in table:
        pytest.skip(f"no oracle digests stored for {name}")
    cfg = table[name]
    ops = synth.NETWORKS[name]()
    images = synth.network_input(cfg["batch"], 224, cfg["seed"])
    net = network.QuantizedNetwork(hq, ops, cfg["seed"], cfg["weight_bits"])
    got = net.build(images, cfg["calib"])
    torch.cuda.synchronize()
    assert set(cfg["tensors"]) == set(got)
    wrong = []
    for key, want in cfg["tensors"].items():
        g = got[key].cpu().numpy()
        h = hashlib.sha256()
        if key == "logits":
            h.update(np.ascontiguousarray(g).tobytes())
        else:
            h.update(np.ascontiguousarray(g[..., :net.chans[key]]).tobytes())
            h.update(net.params[key].tobytes())
        if h.hexdigest() != want:
            wrong.append(key)
    assert not wrong, f"{len(wrong)} of {len(cfg['tensors'])} tensors differ, first: {wrong[:3]}"
    # the timed pass (fused schedule, outputs overwritten in place) reproduces every tensor it writes
    for key, tsr in got.items():
        if key != "in":
            tsr.zero_()
    net.forward()
    torch.cuda.synchronize()
    wrong = []
    for key, want in cfg["tensors"].items():
        if key in net.fused_away or key == "in":
            continue
        g = got[key].cpu().numpy()
        h = hashlib.sha256()
        if key == "logits":
            h.update(np.ascontiguousarray(g).tobytes())
        else:
            h.update(np.ascontiguousarray(g[..., :net.chans[key]]).tobytes())
            h.update(net.params[key].tobytes())
        if h.hexdigest() != want:
            wrong.append(key)
    assert not wrong, f"timed pass: {len(wrong)} tensors differ, first: {wrong[:3]}"
    rc, site = hq.device_status()
    assert rc == 0, (rc, site)
