#!/usr/bin/env python
"""Benchmark of the quantized-convolution hot path on B200.

Workload (default): the quantized GEMM sweep -- uint8 A (MxK) times uint8 B (KxN), both
asymmetric per layer with zero points in [0,255], int32 bias, uint8 output, M=N=K in
{512, 1024, 2048, 4096, 8192}.  One step = one pass over the five sizes through
qtz_conv2d_u8 (activation-sum pre-pass + tcgen05 implicit-GEMM kernel with the fused
zero-point / requantize epilogue).  Metric: int8 TOP/s, 2 ops per multiply-accumulate of the
method itself (no padding, no cross-term work counted).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line on rank 0.  With --impl reference the CPU oracle is timed instead
(a deliberately plain program: a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1806_08342_b200 import synth  # noqa: E402

SIZES = synth.GEMM_SIZES
METRIC, UNIT = "int8_tops", "TOP/s"
WORKLOAD = "quantized GEMM sweep u8xu8 asymmetric, M=N=K in {512,1024,2048,4096,8192}, int32 bias, u8 out"


def step_ops(sizes=None):
    return float(sum(2.0 * s * s * s for s in (SIZES if sizes is None else sizes)))


# DRAM traffic of the dominant kernel: read from the text summary of one ncu capture of the five
# conv_tc_kernel launches of a step (dram__bytes_read.sum + dram__bytes_write.sum, divided by five), which
# also records the SHA-256 of the kernel's sources at the time.  Reported only while those sources are
# unchanged; null otherwise.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "conv_tc_kernel_gemm_sweep_traffic.txt")
TRAFFIC_SOURCES = ("paper_1806_08342_b200/csrc/qtz_conv_tc.cu", "paper_1806_08342_b200/csrc/qtz_ptx.cuh")


def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def kernel_traffic():
    try:
        rec = dict(line.split(":", 1) for line in open(TRAFFIC_FILE) if ":" in line and not line.startswith("#"))
        if rec["kernel_sources_sha256"].strip() != kernel_sources_sha256() or len(SIZES) != 5:
            return None
        return float(rec["dram_bytes_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


# Integer-issue ceiling of the depthwise kernel, in outputs per clock and SM: per output three dp4a (64 lanes
# per clock and SM) and one 32x32->64 multiply-add (16 lanes per clock and SM) on the same pipe:
# 1 / (3/64 + 1/16).  A loop of exactly these instructions measured 9.6.
DW_ALU_OUT_PER_CLK_SM = 1.0 / (3.0 / 64.0 + 1.0 / 16.0)



def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None
        self.nvml, self.samples, self.stop_flag, self.thread = None, [], False, None

    def _poll(self):
        """NVML polled from a thread: (SM MHz, max SM MHz, clock-event reason bits) per sample."""
        nv, dev = self.nvml
        try:
            top = nv.nvmlDeviceGetMaxClockInfo(dev, nv.NVML_CLOCK_SM)
        except Exception:
            top = 0
        while not self.stop_flag:
            try:
                self.samples.append((nv.nvmlDeviceGetClockInfo(dev, nv.NVML_CLOCK_SM), top,
                                     nv.nvmlDeviceGetCurrentClocksEventReasons(dev)))
            except Exception:
                break
            time.sleep(0.001)

    def start(self):
        # the timed region of the default run lasts a few milliseconds: poll NVML directly where it is available
        # (same counters as nvidia-smi's clocks.sm / clocks_event_reasons), else fall back to nvidia-smi at 100 ms
        try:
            import pynvml as nv
            nv.nvmlInit()
            idx = self.index
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            if vis and all(v.strip().isdigit() for v in vis.split(",")) and idx < len(vis.split(",")):
                idx = int(vis.split(",")[idx])
            dev = nv.nvmlDeviceGetHandleByIndex(idx)
            nv.nvmlDeviceGetCurrentClocksEventReasons(dev)
            self.nvml = (nv, dev)
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def count(self):
        return len(self.samples) if self.nvml is not None else len(self.lines)

    def stop(self):
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=1.0)
            nv = self.nvml[0]
            names = (("hw_slowdown", getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8)),
                     ("hw_thermal_slowdown", getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40)),
                     ("sw_thermal_slowdown", getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20)),
                     ("sw_power_cap", getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)))
            reasons = sorted({n for _, _, bits in self.samples for n, mask in names if bits & mask})
            busy = [c for c, _, _ in self.samples if c > 0]
            return {"sm_mhz": float(np.median(busy)) if busy else None,
                    "sm_max_mhz": float(max(m for _, m, _ in self.samples)) if self.samples else None,
                    "reasons": reasons, "samples": len(self.samples), "source": "nvml polled back to back"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [v for v in sm if v > 0]
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# CPU oracle leg
# ------------------------------------------------------------------------------------------
def oracle_sample(rows_per_size, seed=2):
    """Runs the oracle on the first `rows` rows of A for each GEMM size; returns (ops, seconds)."""
    import oracle
    ops, secs = 0.0, 0.0
    for size, rows in rows_per_size.items():
        if rows <= 0:
            continue
        t = synth.gemm_u8(rows, size, size, seed)
        bt = np.ascontiguousarray(t["b"].T).reshape(size, 1, 1, size).astype(np.int32)
        a = t["a"].reshape(rows, 1, 1, size)
        zw = np.full(size, t["z_b"], np.int32)
        m, r = oracle.quantize_multiplier(1e-6)
        mult, rsh = np.full(size, m, np.int32), np.full(size, r, np.int32)
        t0 = time.perf_counter()
        acc = oracle.conv2d_acc(a, t["z_a"], bt, zw, t["bias"], 1, 0)
        oracle.requantize(acc, mult, rsh, 128, 0, 255)
        secs += time.perf_counter() - t0
        ops += 2.0 * rows * size * size
    return ops, secs


def cpu_baseline(target_seconds=15.0):
    import oracle
    oracle.build()
    probe = {SIZES[-1]: 32}
    ops, secs = oracle_sample(probe)
    rate = ops / max(secs, 1e-9)
    budget_ops = rate * target_seconds
    # same row fraction of every size, so the sample has the sweep's mix of shapes
    frac = min(1.0, budget_ops / step_ops())
    rows = {s: max(1, int(round(s * frac))) for s in SIZES}
    ops, secs = oracle_sample(rows)
    cores = oracle.num_threads()
    # the same program on one thread, on a sample a sixth as long
    oracle.set_num_threads(1)
    rows1 = {s: max(1, int(round(s * frac / (6.0 * cores)))) for s in SIZES}
    ops1, secs1 = oracle_sample(rows1)
    oracle.set_num_threads(cores)
    return {"value": ops / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "first rows of A per size " + json.dumps({str(k): v for k, v in rows.items()}) +
                      f" against full B ({ops / 1e9:.1f} GOP in {secs:.1f} s)",
            "one_thread": {"value": ops1 / secs1 / 1e12, "unit": UNIT,
                           "sample": f"{ops1 / 1e9:.1f} GOP in {secs1:.1f} s, rows " + json.dumps({str(k): v for k, v in rows1.items()})}}


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle
    oracle.build()
    probe_ops, probe_s = oracle_sample({8192: 4})
    rate = probe_ops / max(probe_s, 1e-9)
    per_step_s = min(8.0, 150.0 / max(1, args.steps + args.warmup))
    frac = min(1.0, rate * per_step_s / step_ops())
    rows = {s: max(1, int(round(s * frac))) for s in SIZES}
    for _ in range(args.warmup):
        oracle_sample(rows)
    ops = secs = 0.0
    for _ in range(args.steps):
        o, s = oracle_sample(rows)
        ops += o; secs += s
    val = ops / secs / 1e12
    sample = "per step: first rows of A per size " + json.dumps({str(k): v for k, v in rows.items()}) + " against full B"
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "int64", "data": "synthetic",
           "config": {"workload": WORKLOAD, "note": "CPU oracle on host cores; bounded row sample of the workload"},
           "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------
# GPU leg
# ------------------------------------------------------------------------------------------
class GemmCase:
    """One size of the sweep, resident in HBM: plan, input, output, host copies for the e2e leg."""

    def __init__(self, hq, qtz, torch, size, seed=2):
        t = synth.gemm_u8(size, size, size, seed)
        self.size = size
        self.z_a, self.z_b = t["z_a"], t["z_b"]
        self.a_host = torch.from_numpy(t["a"].reshape(size, 1, 1, size)).pin_memory()
        self.a = self.a_host.cuda()
        bt = torch.from_numpy(np.ascontiguousarray(t["b"].T)).cuda()         # OHWI view of B
        bias = torch.from_numpy(t["bias"]).cuda()
        # output quantizer: range of the accumulators, measured with the library itself
        raw = hq.conv_create(qtz.conv_desc(size, 1, 1, size, size, 1, 1, 1, 0, qtz.W_U8_PER_LAYER_ASYM,
                                           qtz.OUT_S32_RAW), bt, bias, self.z_b)
        acc = raw(self.a, self.z_a)
        unit = np.zeros(1, qtz.QPARAMS); unit["scale"] = 1.0
        lo, hi = hq.minmax(hq.dequantize(acc.view(-1), unit))
        raw.close(); del acc
        m, r = qtz.quantize_multiplier(127.0 / (max(abs(float(lo[0])), abs(float(hi[0]))) + 1.0))
        self.plan = hq.conv_create(qtz.conv_desc(size, 1, 1, size, size, 1, 1, 1, 0, qtz.W_U8_PER_LAYER_ASYM),
                                   bt, bias, self.z_b, np.full(size, m, np.int32), np.full(size, r, np.int32))
        self.y = self.plan.empty_output("cuda")
        self.y_host = torch.empty(self.y.shape, dtype=torch.uint8).pin_memory()
        self.ops = 2.0 * size ** 3

    def run(self):
        self.plan(self.a, self.z_a, 128, 0, 255, out=self.y)


def time_hbm_kernels(hq, qtz, torch, peaks):
    """Achieved GB/s of the element-wise and depthwise kernels (algorithmic bytes / event time)."""
    res = {}
    hq_sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    n = 1 << 28                                                    # 1 GiB of fp32: far larger than L2
    x = torch.empty(n, dtype=torch.float32, device="cuda").uniform_(-1.0, 6.0)
    p = hq.calibrate_minmax(x)
    q = hq.quantize_tensor(x, p)

    def timed(fn, reps=5):
        fn(); torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(reps):
            fn()
        e.record(); torch.cuda.synchronize()
        return s.elapsed_time(e) / reps * 1e-3

    def entry(name, secs, nbytes):
        gbs = nbytes / secs / 1e9
        res[name] = {"GB/s": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 3),
                     "ms": round(secs * 1e3, 4)}

    entry("minmax_f32 (4 B/elem)", timed(lambda: hq.minmax(x)), 4.0 * n)
    entry("quantize_f32_to_u8 (5 B/elem)", timed(lambda: hq.quantize_tensor(x, p, out=q)), 5.0 * n)
    entry("dequantize_u8_to_f32 (5 B/elem)", timed(lambda: hq.dequantize(q, p, out=x)), 5.0 * n)
    y = torch.empty_like(x)
    entry("simquant_f32 (8 B/elem)", timed(lambda: hq.simquant(x, p, out=y)), 8.0 * n)
    p16 = hq.calibrate_minmax(x, bits=16)
    q16 = hq.quantize_tensor(x, p16, out_dtype=qtz.U16)
    entry("quantize_f32_to_u16 (6 B/elem)", timed(lambda: hq.quantize_tensor(x, p16, out_dtype=qtz.U16, out=q16)), 6.0 * n)
    entry("dequantize_u16_to_f32 (6 B/elem)", timed(lambda: hq.dequantize(q16, p16, out=y)), 6.0 * n)
    del x, q, y, q16
    # MobileNet-v1 depthwise layers at batch 128: (H, C, stride, zero points and clamp).  "ranged": z_x = 3,
    # z_y = 10, clamp [10,255] (border cells refilled with z_x, explicit clamp); "relu6": the case between two
    # ReLU6 tensors, z_x = z_y = 0 and the whole byte as the range.  At stride 1 the kernel is bound by integer
    # issue, not by HBM: frac_of_alu_peak refers to DW_ALU_OUT_PER_CLK_SM at the SM clock sampled under load.
    for hh, c, stride, name, z in [(112, 64, 2, "ranged", (3, 10, 10, 255)), (56, 128, 1, "ranged", (3, 10, 10, 255)),
                                   (56, 128, 1, "relu6", (0, 0, 0, 255)), (14, 512, 1, "ranged", (3, 10, 10, 255))]:
        xin = torch.randint(0, 256, (128, hh, hh, c), dtype=torch.uint8, device="cuda")
        w = torch.randint(-127, 128, (3, 3, c), dtype=torch.int8, device="cuda")
        m, r = qtz.quantize_multiplier(1.0 / 600.0)
        plan = hq.conv_create(qtz.conv_desc(128, hh, hh, c, c, 3, 3, stride, 1), w, None, None,
                              np.full(c, m, np.int32), np.full(c, r, np.int32), depthwise=True)
        y = plan.empty_output("cuda")
        secs = timed(lambda: plan(xin, *z, out=y), reps=10)
        # the SM clock while this kernel runs, sampled over a longer loop of the same launch
        sampler = ClockSampler(torch.cuda.current_device())
        sampler.start()
        t_end = time.time() + 0.7
        while time.time() < t_end:
            for _ in range(50):
                plan(xin, *z, out=y)
            torch.cuda.synchronize()
        clk = sampler.stop()
        mhz = clk["sm_mhz"] or clk["sm_max_mhz"] or 1965.0
        alu_peak = hq_sms * DW_ALU_OUT_PER_CLK_SM * mhz * 1e6            # outputs per second
        key = f"depthwise3x3 128x{hh}x{hh}x{c} s{stride} {name}"
        entry(key, secs, float(xin.numel() + y.numel()))
        res[key]["frac_of_alu_peak"] = round(y.numel() / secs / alu_peak, 3)
        res[key]["sm_mhz"] = mhz
        plan.close()
    res["requant_alu_probe (outputs per clock and SM)"] = {
        "three_dp4a": round(hq.probe_requant_rate(0)[0], 2), "multiply_shift_clamp": round(hq.probe_requant_rate(1)[0], 2),
        "both": round(hq.probe_requant_rate(2)[0], 2), "derived_ceiling_used": round(DW_ALU_OUT_PER_CLK_SM, 2)}
    a = torch.randint(0, 256, (1 << 28,), dtype=torch.uint8, device="cuda").view(-1, 64)
    b = torch.randint(0, 256, (1 << 28,), dtype=torch.uint8, device="cuda").view(-1, 64)
    ma, mb, r = qtz.add_params(0.02, 0.03, 0.04)
    out = torch.empty_like(a)
    entry("add_u8 (3 B/elem)", timed(lambda: hq.add_u8(a, 3, ma, b, 5, mb, r, 0, 0, 255, 64, out=out)), 3.0 * a.numel())
    return res


def time_layer(hq, qtz, torch, spec, reps=20):
    """One convolution layer alone: spec = "batch,h,w,c,n,k,stride[,dw][,full]" (profiling runs).
    "full" = the zero points and clamp of a layer between two ReLU6 tensors (z_x = z_y = 0, clamp to
    [0,255]); without it z_x = 7, z_y = 20 and the clamp is [20,255]."""
    v = spec.split(",")
    b, hh, ww, c, n, k, st = (int(x) for x in v[:7])
    dw = "dw" in v[7:]
    zargs = (0, 0, 0, 255) if "full" in v[7:] else (7, 20, 20, 255)
    pad = k // 2
    x = torch.randint(0, 256, (b, hh, ww, (c + 15) // 16 * 16), dtype=torch.uint8, device="cuda")
    w = torch.randint(-127, 128, (k, k, c) if dw else (n, k, k, c), dtype=torch.int8, device="cuda")
    m, r = qtz.quantize_multiplier(1.0 / (40.0 * (k * k * (1 if dw else c)) ** 0.5 * 73.0))
    plan = hq.conv_create(qtz.conv_desc(b, hh, ww, c, n, k, k, st, pad), w, None, None, np.full(n, m, np.int32),
                          np.full(n, r, np.int32), depthwise=dw)
    y = plan.empty_output("cuda")
    for _ in range(3):
        plan(x, *zargs, out=y)
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(reps):
        plan(x, *zargs, out=y)
    e.record(); torch.cuda.synchronize()
    ms = s.elapsed_time(e) / reps
    oh, ow = plan.oh, plan.ow
    macs = b * oh * ow * n * k * k * (1 if dw else c)
    nbytes = b * hh * ww * c + b * oh * ow * n
    return {"layer": spec, "kernel": plan.kernel, "detail": plan.detail, "ms": round(ms, 4), "TOP/s": round(2 * macs / ms / 1e9, 1),
            "GB/s": round(nbytes / ms / 1e6, 1), "distinct_outputs": int(torch.unique(y[..., :n]).numel())}


def time_block(hq, qtz, torch, spec, reps=20):
    """One depthwise-separable block: spec = "batch,h,c,n,stride" (3x3 depthwise on h x h x c, then 1x1 to n channels,
    both between ReLU6 tensors).  Times the depthwise kernel, the pointwise kernel, the two in a row and the fused
    call qtz_conv2d_dw_pw_u8, each as a CUDA-graph replay of `reps` launches (profiling runs)."""
    b, hh, c, n, stride = (int(v) for v in spec.split(","))
    x = torch.randint(0, 256, (b, hh, hh, (c + 15) // 16 * 16), dtype=torch.uint8, device="cuda")
    wd = torch.randint(-127, 128, (3, 3, c), dtype=torch.int8, device="cuda")
    m, r = qtz.quantize_multiplier(1.0 / 600.0)
    dw = hq.conv_create(qtz.conv_desc(b, hh, hh, c, c, 3, 3, stride, 1), wd, None, None, np.full(c, m, np.int32),
                        np.full(c, r, np.int32), depthwise=True)
    wp = torch.randint(-127, 128, (n, 1, 1, c), dtype=torch.int8, device="cuda")
    m2, r2 = qtz.quantize_multiplier(1.0 / (40.0 * c ** 0.5 * 73.0))
    pw = hq.conv_create(qtz.conv_desc(b, dw.oh, dw.ow, c, n, 1, 1, 1, 0), wp, None, None, np.full(n, m2, np.int32),
                        np.full(n, r2, np.int32))
    mid, y, y2 = dw.empty_output("cuda"), pw.empty_output("cuda"), pw.empty_output("cuda")

    def replayed(fn):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for _ in range(reps):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        g.replay(); torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(5):
            g.replay()
        e.record(); torch.cuda.synchronize()
        return round(s.elapsed_time(e) / (5 * reps) * 1e3, 1)

    out = {"block": spec,
           "depthwise_us": replayed(lambda: dw(x, 0, 0, 0, 255, out=mid)),
           "pointwise_us": replayed(lambda: pw(mid, 0, 0, 0, 255, out=y)),
           "both_us": replayed(lambda: (dw(x, 0, 0, 0, 255, out=mid), pw(mid, 0, 0, 0, 255, out=y)))}
    try:
        out["fused_us"] = replayed(lambda: pw.after_depthwise(dw, x, 0, 0, 0, 255, 0, 0, 255, out=y2))
        out["fused_equals_both"] = bool(torch.equal(y, y2))
        out["fused_kernel"] = pw.detail
    except qtz.QtzError as exc:
        out["fused_us"], out["fused_kernel"] = None, str(exc)
    return out


NETWORK_CONFIGS = [("mobilenet_v1", 128, 8), ("resnet50", 256, 8), ("mobilenet_v2_14", 256, 4)]


def roofline_sum_ms(ops, batch, wbits, peaks, resolution=224):
    """Lower bound of one forward pass with one kernel per layer and no fusion between layers: per layer the
    larger of its tensor time (dense layers; 2 ops per multiply-accumulate against the int8 peak, taken as the
    measured bf16 burst x 2) and its HBM time (input + output + weights once, against the measured copy rate)."""
    shape = {"in": (resolution, resolution, 3)}
    hbm, tensor = peaks["hbm_gbs"] * 1e9, 2.0 * peaks["bf16_burst"] * 1e12
    total = 0.0
    for op in ops:
        kind = op["op"]
        if kind in ("conv", "fc"):
            h, w, c = shape[op["src"]] if kind == "conv" else (1, 1, op["cin"])
            k, st, pad = (op["k"], op["stride"], op["pad"]) if kind == "conv" else (1, 1, 0)
            oh, ow = (h + 2 * pad - k) // st + 1, (w + 2 * pad - k) // st + 1
            dw = kind == "conv" and op["depthwise"]
            n = op["cout"]
            macs = batch * oh * ow * n * k * k * (1 if dw else op["cin"])
            wbytes = k * k * op["cin"] * (1 if dw else n) * wbits / 8.0
            nbytes = batch * h * w * c + batch * oh * ow * n * (4 if kind == "fc" else 1) + wbytes
            total += max(nbytes / hbm, 0.0 if dw else 2.0 * macs / tensor)
            shape[op["dst"]] = (oh, ow, n)
        elif kind == "add":
            h, w, c = shape[op["a"]]
            total += 3.0 * batch * h * w * c / hbm
            shape[op["dst"]] = (h, w, c)
        elif kind == "maxpool":
            h, w, c = shape[op["src"]]
            oh, ow = (h + 2 * op["pad"] - op["k"]) // op["stride"] + 1, (w + 2 * op["pad"] - op["k"]) // op["stride"] + 1
            total += batch * (h * w + oh * ow) * c / hbm
            shape[op["dst"]] = (oh, ow, c)
        else:
            h, w, c = shape[op["src"]]
            total += batch * (h * w + 1) * c / hbm
            shape[op["dst"]] = (1, 1, c)
    return total * 1e3


def time_networks(hq, qtz, torch, peaks, reps=10, detail=False, only=""):
    """Images/s of whole-network integer inference at the batch sizes of the network workloads
    (calibration and plan creation outside the timed region; activations stay in HBM)."""
    from paper_1806_08342_b200 import network
    res = {}
    for name, batch, wbits in NETWORK_CONFIGS:
        if only and name not in only.split(","):
            continue
        ops = synth.NETWORKS[name]()
        images = synth.network_input(batch, 224, 12)
        net = network.QuantizedNetwork(hq, ops, 12, wbits)
        net.build(images, 2)
        for _ in range(3):
            net.forward()
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(reps):
            net.forward()
        e.record(); torch.cuda.synchronize()
        eager_ms = s.elapsed_time(e) / reps
        # the same pass replayed from a CUDA graph (no host launch gaps)
        graph_ms = None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                net.forward()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    net.forward()
            torch.cuda.current_stream().wait_stream(side)
            g.replay(); torch.cuda.synchronize()
            s.record()
            for _ in range(reps):
                g.replay()
            e.record(); torch.cuda.synchronize()
            graph_ms = s.elapsed_time(e) / reps
        except Exception as exc:  # graph capture is an optimisation of the harness, not of the library
            graph_ms = None
            res.setdefault("graph_errors", []).append(f"{name}: {type(exc).__name__}: {exc}"[:200])
        best = min(eager_ms, graph_ms) if graph_ms else eager_ms
        bound = roofline_sum_ms(ops, batch, wbits, peaks)
        entry = {"batch": batch, "weight_bits": wbits, "ms_eager": round(eager_ms, 4),
                 "ms_graph": None if graph_ms is None else round(graph_ms, 4), "images_per_s": round(batch / best * 1e3, 1),
                 "roofline_sum_ms": round(bound, 4), "frac_of_roofline_sum": round(bound / best, 3),
                 "launches": net.num_launch_calls()}
        if detail:
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(net.schedule) + 1)]
            t = net.tensors
            evs[0].record()
            for i, item in enumerate(net.schedule):
                net.run_item(item)
                evs[i + 1].record()
            torch.cuda.synchronize()
            rows = []
            for i, item in enumerate(net.schedule):
                L = item[2] if item[0] == "conv+add" else item[1]
                kern = item[1].plan.detail if item[0] in ("conv", "fc", "conv+add", "dw+pw") else item[0]
                rows.append((round(evs[i].elapsed_time(evs[i + 1]) * 1e3, 1), L.op.get("dst"), kern,
                             tuple(t[L.op["dst"]].shape)))
            entry["layers_us"] = rows
        res[name] = entry
        del net
        torch.cuda.empty_cache()
    return res


def probe_int8(hq, torch, device_index, sustained_seconds=4.0):
    """tcgen05.mma kind::i8 alone (operands resident in shared memory, nothing loaded in the loop): a burst figure
    (ten launches of about 1 ms) and one held for `sustained_seconds` with the SM clock sampled meanwhile."""
    hq.probe_int8_peak(8192, 2)                                       # warm-up, module load
    burst = max(hq.probe_int8_peak(16384, 10)[0] for _ in range(3))
    sampler = ClockSampler(device_index)
    sampler.start()
    t0, ops_t, ms_t = time.time(), 0.0, 0.0
    while time.time() - t0 < sustained_seconds:
        tops, ms = hq.probe_int8_peak(16384, 100)
        ops_t += tops * ms
        ms_t += ms
    clocks = sampler.stop()
    return {"burst_tops": round(burst, 1), "sustained_tops": round(ops_t / ms_t, 1), "sustained_seconds": round(ms_t * 1e-3, 2),
            "clocks_sustained": clocks, "how": "128x256x32 u8*s8->s32 MMAs back to back on shared-memory resident operands, one CTA per SM"}


def sustained_gemm(case, torch, device_index, seconds=2.5):
    """The largest size of the sweep back to back for `seconds`, with the SM clock sampled meanwhile."""
    sampler = ClockSampler(device_index)
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        case.run()
    torch.cuda.synchronize()
    sampler.start()
    t0, n, ms = time.time(), 0, 0.0
    while time.time() - t0 < seconds:
        s.record()
        for _ in range(200):
            case.run()
        e.record(); torch.cuda.synchronize()
        ms += s.elapsed_time(e); n += 200
    clocks = sampler.stop()
    return {"size": case.size, "launches": n, "seconds": round(ms * 1e-3, 2), "TOP/s": round(case.ops * n / (ms * 1e-3) / 1e12, 1),
            "clocks": clocks, "includes": "pixel_sum_kernel pre-pass + conv_tc_kernel per launch"}


def max_over_ranks(values, dist, device):
    """The slowest rank's value of each entry (device-timed durations): replicas run side by side and the
    job is done when the last one is."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(ops_per_rank_step, steps, world, ms):
    """Aggregate throughput of `world` replicas (weak scaling: every rank does the full step)."""
    return world * ops_per_rank_step * steps / (ms * 1e-3) / 1e12


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_1806_08342_b200 import build as qbuild
    qbuild.build()
    from paper_1806_08342_b200 import qtz

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    hq = qtz.Handle(local_rank)
    if args.probe_int8:
        print(json.dumps({"int8_probe": probe_int8(hq, torch, local_rank)}), flush=True)
        return
    if args.hbm_only:
        print(json.dumps({"hbm_kernels": time_hbm_kernels(hq, qtz, torch, peaks)}), flush=True)
        return
    if args.layer:
        print(json.dumps({"layers": [time_layer(hq, qtz, torch, sp) for sp in args.layer.split(";")]}), flush=True)
        return
    if args.block:
        print(json.dumps({"blocks": [time_block(hq, qtz, torch, sp) for sp in args.block.split(";")]}), flush=True)
        return
    if args.networks_only:
        print(json.dumps({"networks": time_networks(hq, qtz, torch, peaks, reps=args.network_reps, detail=True,
                                                    only=args.networks)}), flush=True)
        return
    cases = [GemmCase(hq, qtz, torch, s) for s in SIZES]
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        for c in cases:
            c.run()
    # The timed region: exactly K steps of plain library calls, nothing else on the stream (consecutive kernels
    # are programmatic dependents of one another, which any stream operation between them would undo).
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for step in range(args.steps):
        for c in cases:
            c.run()
    t1.record()
    barrier()
    in_region = sampler.count()      # the sampler keeps running over the two passes below: the same launches again
    ms = t0.elapsed_time(t1)
    # The same K steps replayed from a CUDA graph of one step (no host launch gaps between the ten kernels).
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for c in cases:
                c.run()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for c in cases:
                    c.run()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            g.replay()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for step in range(args.steps):
            g.replay()
        g1.record()
        barrier()
        graph_ms = g0.elapsed_time(g1)
    except Exception as exc:   # capture is a convenience of the harness, not of the library
        graph_ms = None
        sys.stderr.write(f"graph replay skipped: {type(exc).__name__}: {exc}\n")
    # The same K steps once more with the library's profiling hook on: CUDA events on the launch stream around every
    # launch of the dominant kernel (and the activation-sum pre-pass it runs beside).  These per-launch durations
    # feed `roofline` and `sweep`; the events between launches cost a little, so this region is not the one timed above.
    kev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in cases]
           for _ in range(args.steps)]
    for row in kev:
        for s, e in row:
            s.record(); e.record()
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for step in range(args.steps):
        for c, (s, e) in zip(cases, kev[step]):
            c.plan.set_profile_events(s, e)
            c.run()
    p1.record()
    barrier()
    ms_profiled = p0.elapsed_time(p1)
    clocks = sampler.stop()
    clocks["samples_in_timed_region"] = in_region
    clocks["window"] = "the timed region and the graph-replay and per-launch-event passes of the same steps after it"
    for c in cases:
        c.plan.set_profile_events(None, None)
    rc, site = hq.device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at site {site}")
    per_size_ms = [float(np.mean([kev[st][i][0].elapsed_time(kev[st][i][1]) for st in range(args.steps)]))
                   for i in range(len(cases))]

    # end to end: host buffers in, host buffers out, every copy inside the timed region.  A user with pinned
    # buffers overlaps the three legs: uploads, kernels and downloads run on a stream each (all library
    # calls stay on ONE stream, as the handle requires) and events order them per tensor -- an input is
    # not overwritten before the kernel that read it is done, an output not before its download is.
    e2e_steps = max(1, min(args.steps, 5))
    cur = torch.cuda.current_stream()
    up, run, down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_pass(steps):
        a_free = [None] * len(cases)
        y_free = [None] * len(cases)
        for _ in range(steps):
            for i, c in enumerate(cases):
                with torch.cuda.stream(up):
                    if a_free[i] is not None:
                        up.wait_event(a_free[i])
                    c.a.copy_(c.a_host, non_blocking=True)
                    a_ready = torch.cuda.Event(); a_ready.record(up)
                with torch.cuda.stream(run):
                    run.wait_event(a_ready)
                    if y_free[i] is not None:
                        run.wait_event(y_free[i])
                    c.run()
                    done = torch.cuda.Event(); done.record(run)
                    a_free[i] = done
                with torch.cuda.stream(down):
                    down.wait_event(done)
                    c.y_host.copy_(c.y, non_blocking=True)
                    y_free[i] = torch.cuda.Event(); y_free[i].record(down)

    def fork():
        ev = torch.cuda.Event(); ev.record(cur)
        for st in (up, run, down):
            st.wait_event(ev)

    def join():
        for st in (up, run, down):
            ev = torch.cuda.Event(); ev.record(st)
            cur.wait_event(ev)

    fork(); e2e_pass(1); join()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fork(); e2e_pass(e2e_steps); join()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    ops = step_ops()
    value = whole_job_value(ops, args.steps, world, ms)
    int8_peak = 2.0 * peaks["bf16_burst"]          # dense int8 : bf16 is 2 : 1 on this part (4.5 vs 2.25 POP/s nominal)
    kernel_tops = ops / (sum(per_size_ms) * 1e-3) / 1e12
    sweep = {str(c.size): {"kernel_ms": round(per_size_ms[i], 4),
                           "TOP/s": round(c.ops / (per_size_ms[i] * 1e-3) / 1e12, 1),
                           "frac_of_int8_peak": round(c.ops / (per_size_ms[i] * 1e-3) / 1e12 / int8_peak, 3)}
             for i, c in enumerate(cases)}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8*s8->s32", "data": "synthetic",
        "config": {"workload": WORKLOAD if len(SIZES) == 5 else WORKLOAD + f" [subset {list(SIZES)}]", "parallelism": f"replicas x{world}",
                   "l2": "operands larger than L2: 268 MB touched per step, 201 MB by the largest size alone",
                   "kernels_per_step": "5 x (pixel_sum_kernel + conv_tc_kernel)",
                   "per_launch_events": f"taken in a second pass of the same {args.steps} steps ({ms_profiled / args.steps:.4f} ms per step with the events)",
                   "graph_replay_ms_per_step": None if graph_ms is None else round(graph_ms / args.steps, 4)},
        "clocks": clocks,
        "e2e": {"value": world * ops * e2e_steps / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": int(sum(c.a_host.numel() for c in cases)),
                "d2h_bytes_per_step": int(sum(c.y_host.numel() for c in cases)), "steps": e2e_steps,
                "how": "pinned host buffers; upload, kernel and download streams overlapped, ordered per tensor by events"},
        "gpu_launches": 2 * len(cases) * args.steps,
        "roofline": {"bound": "tensor", "kernel": "conv_tc_kernel", "achieved": kernel_tops, "peak": int8_peak,
                     "unit": UNIT, "frac": kernel_tops / int8_peak, "traffic": kernel_traffic(),
                     "traffic_unit": "bytes per launch (algorithmic: 53.7e6)",
                     "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_burst']} TFLOP/s x 2 (int8:bf16 nominal ratio)",
                     "frac_of_sustained_peak": kernel_tops / (2.0 * peaks["bf16_sustained"]),
                     "frac_of_nominal_4500": kernel_tops / 4500.0},
        "sweep": sweep,
    }
    if world == 1 and not args.no_extras:
        probe = probe_int8(hq, torch, local_rank, sustained_seconds=3.0)
        out["roofline"]["int8_peak_measured"] = probe
        out["roofline"]["frac_of_int8_measured_burst"] = kernel_tops / probe["burst_tops"]
        sus = sustained_gemm(cases[-1], torch, local_rank)
        sus["frac_of_sustained_peak"] = round(sus["TOP/s"] / (2.0 * peaks["bf16_sustained"]), 3)
        sus["frac_of_int8_measured_sustained"] = round(sus["TOP/s"] / probe["sustained_tops"], 3)
        out["sustained"] = sus
        out["hbm_kernels"] = time_hbm_kernels(hq, qtz, torch, peaks)
        out["networks"] = time_networks(hq, qtz, torch, peaks)
        out["cpu_baseline"] = cpu_baseline()
    print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the HBM-kernel table and the CPU baseline")
    ap.add_argument("--probe-int8", action="store_true",
                    help="run only the tensor-core probe (tcgen05.mma kind::i8, burst and 4-s sustained); prints it as JSON")
    ap.add_argument("--hbm-only", action="store_true",
                    help="run only the element-wise / depthwise kernel table (profiling runs); prints it as JSON")
    ap.add_argument("--layer", default="", help='time single conv layers: "batch,h,w,c,n,k,stride[,dw];..." (profiling runs)')
    ap.add_argument("--block", default="", help='time depthwise-separable blocks, separate and fused: "batch,h,c,n,stride;..." (profiling runs)')
    ap.add_argument("--networks-only", action="store_true",
                    help="run only the whole-network timings, with per-layer times; prints them as JSON")
    ap.add_argument("--networks", default="", help="with --networks-only: comma-separated subset of the networks (profiling runs)")
    ap.add_argument("--network-reps", type=int, default=10, help="with --networks-only: timed passes per network")
    ap.add_argument("--sizes", default="", help="comma-separated subset of the sweep (profiling runs); default: all")
    args = ap.parse_args()
    if args.sizes:
        global SIZES
        SIZES = tuple(int(v) for v in args.sizes.split(","))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
