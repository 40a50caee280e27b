#!/usr/bin/env python
"""Writes tests/golden/network_hashes.json: SHA-256 of every tensor of the three network workloads at
their full batch sizes, computed by the CPU oracle alone (oracle/netrun.py; nothing of the CUDA
library is imported or run).

    python tests/golden/make_network_hashes.py [network ...]

Inputs are the seeded synthetic images of synth.network_input(batch, 224, seed) with the quantizers
calibrated on the first `calib` images (Section 3.1.2).  A tensor is hashed as the bytes of its codes
[B,H,W,C] in C order without channel padding (the int32 logits as [B,classes]), followed by the
16-byte quantizer record when it has one.  The GPU test recomputes the same digests from the
library's output (tests/test_gpu_networks.py::test_network_full_batch_every_image).
Takes a few minutes for MobileNet-v1/v2 and about a quarter of an hour for ResNet-50 on 8 cores.
"""
import hashlib
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from oracle import netrun  # noqa: E402
from paper_1806_08342_b200 import synth  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "network_hashes.json")
# network -> (batch, weight bits, seed, calibration images): the launch configurations the benchmark times
CONFIGS = {"mobilenet_v1": (128, 8, 12, 2), "resnet50": (256, 8, 12, 2), "mobilenet_v2_14": (256, 4, 12, 2)}


def digest(q, p):
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(q).tobytes())
    if p is not None:
        h.update(p.tobytes())
    return h.hexdigest()


def main():
    names = sys.argv[1:] or list(CONFIGS)
    table = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for name in names:
        batch, wbits, seed, calib = CONFIGS[name]
        images = synth.network_input(batch, 224, seed)
        entry = {"batch": batch, "weight_bits": wbits, "seed": seed, "calib": calib, "tensors": {}}
        t0 = time.time()
        netrun.run(synth.NETWORKS[name](), images, calib, seed, wbits,
                   visit=lambda key, t: entry["tensors"].__setitem__(key, digest(t.q, t.p)), keep=False)
        entry["oracle_seconds"] = round(time.time() - t0, 1)
        table[name] = entry
        with open(OUT, "w") as f:
            json.dump(table, f, indent=1, sort_keys=True)
        print(name, len(entry["tensors"]), "tensors", entry["oracle_seconds"], "s", flush=True)


if __name__ == "__main__":
    main()
