"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The data path has no collective (replicas
only); what ranks exchange is the timing reduction, and the reference arm runs on rank 0 alone."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["QTZ_ROOT"])
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
# each rank "measured" its own durations; the job takes as long as the slowest replica
ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 40.0 - 3.0 * rank], dist, "cpu")
value = bench.whole_job_value(2.0e12, 4, world, ms)
dist.barrier()
print(json.dumps({"rank": rank, "ms": ms, "e2e": e2e, "value": value}), flush=True)
dist.destroy_process_group()
"""


def test_timing_reduction_is_max_over_ranks_and_work_is_summed():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   QTZ_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", _WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 15.0 and o["e2e"] == 40.0                  # the slowest rank of each entry
        assert abs(o["value"] - 2 * 2.0e12 * 4 / 15.0e-3 / 1e12) < 1e-9   # both replicas' work over that time


@pytest.mark.timeout(300)
def test_reference_arm_runs_on_rank_zero_only():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="4")
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                                       "--steps", "1", "--warmup", "0", "--sizes", "512"], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    out0, err0 = procs[0].communicate(timeout=280)
    out1, err1 = procs[1].communicate(timeout=280)
    assert procs[0].returncode == 0, err0[-2000:]
    assert procs[1].returncode == 0 and out1.strip() == ""          # the other rank leaves without work
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
