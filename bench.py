#!/usr/bin/env python
"""Benchmark of the quantized-convolution path on B200.

A step is one int8 inference pass of a whole network-shaped stack over one batch: input
conversion (float -> int8), every convolution with its fused epilogue, and the max-pools,
replayed as one CUDA graph.  Calibration (statistics + exponent choice) runs once before the
timed region, as the method prescribes, and is timed separately.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50|vgg16|inception|mobilenet]
  python bench.py --impl reference ...      # the CPU oracle on the host cores (slow on purpose)

Prints one JSON line (rank 0).  The headline (`value`, `ms_per_step`, `config`) is the ResNet-50-shaped
stack; with one GPU and no --workload the line also carries, under `workloads`, the other three stacks,
the single-layer configuration, the calibration-statistics call and the tensor pipe's measured int8
ceiling.  With --per-layer a table goes to stderr.
"""
import argparse
import hashlib
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1805_07941_b200 import workloads as wl  # noqa: E402

WORKLOADS = {
    "resnet50": (lambda: wl.resnet50(batch=32), "ResNet-50-shaped int8 conv stack, batch 32, 224x224x3"),
    "vgg16": (lambda: wl.vgg16(batch=64), "VGG-16-shaped int8 conv layers, batch 64, 224x224x3"),
    "inception": (lambda: wl.inception(batch=128), "GoogLeNet-style inception blocks, batch 128, 28x28x192"),
    "mobilenet": (lambda: wl.mobilenet(batch=256), "MobileNet-v1-shaped int8 network, batch 256, 224x224x3"),
}
METRIC = "int8 conv images/sec (whole stack, 1 B200); TOPS and roofline fraction alongside"
NOMINAL_INT8_TOPS = 4500.0          # dense, public datasheet figure
NOMINAL_HBM_GBS = 8000.0
MMA_MACS_PER_CLK_PER_SM = 8192.0    # a 128x128x32 kind::i8 instruction per 64 SM clocks (measured: --mma-peak)


def measured_peaks():
    """HBM GB/s and dense bf16 TFLOP/s measured on this machine (generated file), else the
    documented fallback.  The int8 tensor peak is the bf16 figure times the nominal ratio 2: the burst
    figure for the millisecond-long steps timed here, the sustained one carried beside it."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def csrc_sha256():
    """Fingerprint of the CUDA sources: a stored DRAM-traffic figure is valid only for the kernels it was taken on."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_1805_07941_b200", "csrc")
    for f in sorted(os.listdir(d)):
        if f.endswith((".cu", ".cuh")):
            with open(os.path.join(d, f), "rb") as fh:
                h.update(fh.read())
    return h.hexdigest()


def stored_traffic(workload):
    """DRAM bytes per launch of the tensor-core kernel from the committed ncu summary, or None when
    there is none for this workload or the CUDA sources have changed since it was taken."""
    import re
    path = os.path.join(ROOT, "profiles", "igemm_traffic_%s.md" % workload)
    if not os.path.exists(path):
        return None
    text = open(path).read()
    m_t = re.search(r"traffic_bytes_per_launch: (\d+)", text)
    m_h = re.search(r"csrc_sha256: ([0-9a-f]+)", text)
    if not m_t or not m_h or m_h.group(1) != csrc_sha256():
        return None
    return int(m_t.group(1))


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, device_index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self.stop_flag.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def result(self):
        self.stop_flag.set()
        if self.ok:
            self.join(timeout=1.0)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_rate(net, weights, x, seconds_target=15.0):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    from oracle import network_ref, ref
    t0 = time.time()
    params, e_buf, _, _ = network_ref.calibrate(net, x[:1], weights)
    t_cal = time.time() - t0
    t0 = time.time()
    network_ref.run(net, x[:1], params, e_buf)
    t1 = time.time() - t0
    n = int(max(1, min(x.shape[0], seconds_target / max(t1, 1e-3))))
    t0 = time.time()
    network_ref.run(net, x[:n], params, e_buf)
    dt = time.time() - t0
    return dict(value=n / dt, unit="img/s", cores=ref.num_threads(), kind="oracle",
                sample="int8 inference of %d image(s) of the batch (calibrated on 1 image in %.1f s)" % (n, t_cal))


def run_reference(args, net, desc):
    """--impl reference: the oracle on the host cores; each step is one image of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import network_ref, ref
    weights = {nd["name"]: wl.gen_weights(nd, 0) for nd in net["nodes"] if nd["op"] == "conv"}
    x = wl.gen_input(net, seed=0, batch=1)
    params, e_buf, _, _ = network_ref.calibrate(net, x, weights)
    for _ in range(args.warmup):
        network_ref.run(net, x, params, e_buf)
    t0 = time.time()
    for _ in range(args.steps):
        network_ref.run(net, x, params, e_buf)
    dt = time.time() - t0
    v = args.steps / dt
    cb = dict(value=v, unit="img/s", cores=ref.num_threads(), kind="oracle",
              sample="each step = int8 inference of 1 image of the batch")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "img/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "config": {"workload": desc, "sample": "1 image per step"},
        "cpu_baseline": cb, "e2e": {"value": v, "unit": "img/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def calib_call(elems, warmup, reps):
    """The calibration-statistics call alone (two passes: maximum, then histogram) on `elems` ReLU-like
    floats, and the threshold search that consumes its histogram (Algorithm 1), host to host."""
    import torch
    from paper_1805_07941_b200 import binding
    x = torch.randn(elems, device="cuda").relu_()
    for _ in range(max(1, warmup)):
        st = binding.qcalib_collect(x, 2048)
    times = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        st = binding.qcalib_collect(x, 2048)
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    ms = float(np.median(times))
    thr = []
    for _ in range(max(1, warmup) + reps):
        t0 = time.perf_counter()
        gamma, delta = binding.qthreshold_search(st["hist"], st["maxabs"], 8, 7, "l1")
        thr.append((time.perf_counter() - t0) * 1e3)
    pk = measured_peaks()
    gbs = 8.0 * elems / ms / 1e6
    del x
    return {"call": "qcalib_collect", "elems": elems, "ms": ms, "maxabs": float(st["maxabs"]),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / pk["hbm_gbs"], "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
                         "bytes": "8 per element: two passes of 4 (maximum, then histogram on [0, maximum])"},
            "note": "whole call: clear, two passes, finalize kernel, two device-to-host copies and the sync",
            "threshold_search": {"gamma": gamma, "delta": delta, "nbins": 2048, "measure": "l1",
                                 "ms_host_to_host": float(np.median(thr[max(1, warmup):]))}}


def single_conv_call(warmup, reps):
    """The one-layer configuration (1x32x32x16 -> 16, 3x3, shift 7, ReLU): 4.7 MOP and 40 KB, so what is
    measured is latency -- device time per launch in a train of launches, and the host-to-host time of
    one call followed by a synchronisation."""
    import torch
    from paper_1805_07941_b200 import binding
    c = wl.single_conv_cfg()
    conv = binding.QConv(c["w"], c["bias"], c["shift"], N=1, H=32, W=32, C=16, K=16, R=3, S=3, pad_h=1, pad_w=1,
                         relu=1, weight_layout=1)
    x = torch.from_numpy(c["x"]).cuda()
    y = torch.empty((1, 32, 32, 16), dtype=torch.int8, device="cuda")
    for _ in range(max(3, warmup)):
        conv.run(x, y)
    torch.cuda.synchronize()
    train = 50
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(2_000_000)                             # the host queues the train behind a busy GPU
    a.record()
    for _ in range(train):
        conv.run(x, y)
    b.record()
    torch.cuda.synchronize()
    host = []
    for _ in range(reps):
        t0 = time.perf_counter()
        conv.run(x, y)
        torch.cuda.synchronize()
        host.append((time.perf_counter() - t0) * 1e6)
    assert conv.status() == 0
    out = {"call": "qconv_run, single-layer configuration (1x32x32x16, 3x3x16x16, shift 7, ReLU)",
           "plan": conv.describe(), "us_per_launch_in_a_train": a.elapsed_time(b) * 1e3 / train,
           "us_host_to_host_median": float(np.median(host)), "ops": 2 * 1024 * 16 * 144,
           "note": "latency-bound: 4.7 MOP and 40 KB per launch"}
    conv.destroy()
    return out


def mma_peak_call():
    """The tensor pipe's own int8 ceiling (MMA train on resident operands), N = 128 and N = 256."""
    from paper_1805_07941_b200 import binding
    out = {}
    for bn in (128, 256):
        r = binding.qbench_mma_i8(bn, 16384)
        out["n%d" % bn] = {"tops": r["tops"], "cycles_per_mma_128xNx32": r["cycles_per_mma"],
                           "macs_per_clk_per_sm": r["macs_per_clk_per_sm"], "ms": r["ms"], "ctas": r["ctas"]}
    return out


def run_single_layer(args, net, desc):
    """--layer NAME: one convolution of the workload, stand-alone, on seeded int8 activations (a
    small, self-contained case for profilers and tile sweeps)."""
    import torch
    from paper_1805_07941_b200 import binding
    nd = [n for n in net["nodes"] if n["name"] == args.layer][0]
    N = args.batch or net["input"][0]
    rng = np.random.default_rng(nd["tid"])
    cg = nd["C"] // nd["groups"]
    x = torch.from_numpy(wl.gen_activation_i8((N, nd["H"], nd["W"], nd["C"]), 0, nd["tid"] + 2)).cuda()
    wq = rng.integers(-128, 128, size=(nd["K"], nd["R"], nd["S"], cg), dtype=np.int8)
    bias = rng.integers(-2**12, 2**12, size=nd["K"]).astype(np.int32)
    shift = np.full(nd["K"], int(np.log2(max(2.0, np.sqrt(nd["R"] * nd["S"] * cg) * 74 * 26 / 48))), np.int32)
    res = t = None
    if nd["residual"]:
        res = torch.from_numpy(wl.gen_activation_i8((N, nd["P"], nd["Q"], nd["K"]), 0, nd["tid"] + 3)).cuda()
        t = (shift - 1).clip(0, 23).astype(np.int32)
    pitch = net["buffers"][nd["dst"]][2]
    conv = binding.QConv(wq, bias, shift, t, None, N=N, H=nd["H"], W=nd["W"], C=nd["C"], K=nd["K"], R=nd["R"],
                         S=nd["S"], stride_h=nd["stride"], stride_w=nd["stride"], pad_h=nd["pad"], pad_w=nd["pad"],
                         groups=nd["groups"], relu=nd["relu"], symmetric=nd["symmetric"],
                         out_c_offset=nd["dst_c_offset"], out_c_pitch=pitch, has_residual=int(res is not None),
                         pool=2 if args.pool else 0)
    y = torch.zeros((N, nd["P"], nd["Q"], pitch), dtype=torch.int8, device="cuda")   # (a pooled layer writes a quarter of it)
    flush = torch.empty(256 << 20, dtype=torch.int8, device="cuda")
    for _ in range(args.warmup):
        conv.run(x, y, res)
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        flush.fill_(1)
        torch.cuda._sleep(400_000)                           # queue the launch behind a busy GPU
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        conv.run(x, y, res)
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    assert conv.status() == 0
    # CUDA events on this system tick in ~2 us steps: also time a train of back-to-back launches
    inner = 20
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(2_000_000)
    a.record()
    for _ in range(inner):
        conv.run(x, y, res)
    b.record()
    torch.cuda.synchronize()
    warm_us = a.elapsed_time(b) * 1e3 / inner
    ms = float(np.median(times))
    ops, byt = 2 * wl.conv_macs(nd, N), wl.conv_alg_bytes(nd, N)
    pk = measured_peaks()
    print(json.dumps({"layer": nd["name"], "workload": desc, "batch": N, "plan": conv.describe(), "us": ms * 1e3, "us_train": warm_us,
                      "us_min": min(times) * 1e3, "tops": ops / ms / 1e9, "gbs": byt / ms / 1e6,
                      "frac_hbm": byt / ms / 1e6 / pk["hbm_gbs"], "frac_int8_burst": ops / ms / 1e9 / (2 * pk["bf16"]),
                      "alg_bytes": byt, "ops": ops}))


def timed_sets(replay, flush, steps, sets):
    """`sets` repetitions of `steps` replays, each replay bracketed by CUDA events after an L2 flush
    (the flush is not timed).  Returns the per-set mean step time in ms."""
    import torch
    out = []
    for _ in range(sets):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in evs:
            flush.fill_(1)
            a.record()
            replay()
            b.record()
        torch.cuda.synchronize()
        out.append(sum(a.elapsed_time(b) for a, b in evs) / steps)
    return out


def measure_network(name, args, rank, world, flush, headline):
    """Calibrate, capture and time one workload.  Returns (result dict, QNetwork, host input)."""
    import torch
    from paper_1805_07941_b200 import binding, dist as qdist
    from paper_1805_07941_b200.network import QNetwork
    make, desc = WORKLOADS[name]
    net = make()
    N = net["input"][0]
    weights = {nd["name"]: wl.gen_weights(nd, 0) for nd in net["nodes"] if nd["op"] == "conv"}
    x_host = wl.gen_input(net, seed=rank)                    # every rank its own batch: weak scaling
    x_pinned = torch.from_numpy(x_host).pin_memory()
    x_dev = x_pinned.cuda()
    qn = QNetwork(net, weights)
    t0 = time.time()
    qn.calibrate(x_dev, sync=world > 1)                      # one calibration batch, split over the ranks
    torch.cuda.synchronize()
    t_cal = time.time() - t0
    qn.check_status()
    if not args.no_graph:
        qn.capture(args.graph_form)                          # None: keeps the fastest of the forms that apply
    qn.x_static.copy_(x_dev)

    def step():
        if qn.graph is not None:
            qn.graph.replay()
        else:
            qn.forward_static()

    convs = [nd for nd in net["nodes"] if nd["op"] == "conv"]
    macs = sum(wl.conv_macs(nd, N) for nd in convs)
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    sets = timed_sets(step, flush, args.steps, args.sets)
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    clocks = sampler.result()
    qn.check_status()
    sets = [qdist.max_over_ranks(s, device="cuda") for s in sets]
    ms_per_step = float(np.median(sets))
    value = world * N / (ms_per_step * 1e-3)

    # Kernels of the step other than the tensor-core one (input conversion, max-pools, depthwise and
    # direct layers), replayed as a graph of their own under the same flush: what is left of the step
    # is the tensor-core kernel's (an upper bound of its time: the others find more in L2 when alone).
    plans = {nd["name"]: qn.handles[nd["name"]].describe() for nd in convs}
    tc = [nd for nd in convs if plans[nd["name"]].startswith("igemm")]
    others = [nd for nd in net["nodes"] if nd["op"] != "conv" or not plans[nd["name"]].startswith("igemm")]
    other_ms = 0.0
    if qn.graph is not None:
        def others_pass():
            qn._convert_input(slice(0, N))
            for nd in others:
                qn._run_node(nd, slice(0, N))
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            others_pass()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g_others = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_others):
            others_pass()
        for _ in range(3):
            g_others.replay()
        other_ms = float(np.median(timed_sets(g_others.replay, flush, args.steps, 3)))
        step()                                               # leave the buffers as a full step leaves them
        torch.cuda.synchronize()
    pk = measured_peaks()
    int8_burst, int8_sust = 2.0 * pk["bf16"], 2.0 * pk["bf16_sustained"]
    mhz = clocks["sm_mhz"] or clocks["sm_max_mhz"] or 1965.0
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    int8_mma = sms * MMA_MACS_PER_CLK_PER_SM * 2.0 * mhz * 1e6 / 1e12          # TOPS at the sampled clock
    tc_ms = max(ms_per_step - other_ms, 1e-6)
    tc_bytes = sum(wl.conv_alg_bytes(nd, N) for nd in tc)
    tc_ops = sum(2 * wl.conv_macs(nd, N) for nd in tc)
    all_bytes = sum(wl.conv_alg_bytes(nd, N) for nd in convs)
    hbm_bound = tc_bytes / (pk["hbm_gbs"] * 1e9) >= tc_ops / (int8_burst * 1e12)
    roof = {"kernel": "igemm_i8_kernel", "bound": "hbm" if hbm_bound else "tensor",
            "launches_per_step": len(tc), "kernel_ms_per_step": tc_ms, "other_kernels_ms_per_step": other_ms,
            "avg_launch_us": 1e3 * tc_ms / max(1, len(tc)),
            "how": "step time (graph replay, CUDA events, L2 flushed before) minus the step's other kernels replayed "
                   "alone under the same flush; algorithmic bytes / ops of the kernel's launches over that time",
            "algorithmic_bytes_per_launch": tc_bytes / max(1, len(tc)),
            "traffic": stored_traffic(name),
            "traffic_note": "ncu DRAM bytes of representative layers scaled to the stack; write-backs that land "
                            "after a kernel's window are not in it (a lower figure than the true traffic)",
            "stack_hbm_frac": all_bytes / (ms_per_step * 1e-3) / 1e9 / pk["hbm_gbs"]}
    if hbm_bound:
        ach = tc_bytes / (tc_ms * 1e-3) / 1e9
        roof.update(achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                    peak_source=pk["source"] + " copy bandwidth", frac_of_nominal_8000=ach / NOMINAL_HBM_GBS)
    else:
        ach = tc_ops / (tc_ms * 1e-3) / 1e12
        roof.update(achieved=ach, peak=int8_burst, unit="TOP/s", frac=ach / int8_burst,
                    peak_source=pk["source"] + " bf16 burst x 2 (nominal int8:bf16 ratio)",
                    frac_of_sustained_x2=ach / int8_sust, frac_of_nominal_4500=ach / NOMINAL_INT8_TOPS,
                    frac_of_mma_rate_at_sampled_clock=ach / int8_mma, mma_rate_peak_tops=int8_mma)
    res = {"workload": desc, "ms_per_step": ms_per_step, "ms_per_step_sets": {"median": ms_per_step, "min": min(sets),
                                                                               "max": max(sets), "n_sets": len(sets)},
           "img_per_s": value, "tops": 2.0 * macs * world / (ms_per_step * 1e-3) / 1e12,
           "graph": qn.graph is not None, "graph_form": getattr(qn, "graph_form", None) if qn.graph is not None else None,
           "graph_forms_tried_ms": getattr(qn, "graph_timings", None), "launches_per_step": qn.num_launches(),
           "roofline": roof, "clocks": clocks, "calibration_s": t_cal}
    if not headline:
        qn.destroy()
        return res, None, None, None, None
    return res, qn, x_host, x_pinned, (net, weights)


def per_layer_table(qn, net, flush):
    """Stand-alone layer times for the --per-layer table: trains of 8 back-to-back launches of one layer
    (CUDA events tick in ~2 us steps, and a lone launch also pays the host's launch latency).  Launches
    2..8 of a train find their operands in L2: the GB/s column is algorithmic bytes over time, not an HBM
    figure, and none of this feeds the JSON line's roofline."""
    import torch
    from paper_1805_07941_b200 import binding
    N = net["input"][0]
    reps, train = 3, 8
    per = {nd["name"]: [] for nd in net["nodes"]}
    for _ in range(reps):
        flush.fill_(1)
        binding.qquantize_f32(qn.x_static, qn.e_buf["input"], 8, out=qn.bufs["input"])
        for nd in net["nodes"]:
            torch.cuda._sleep(600_000)                       # hold the GPU while the host queues the train
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(train):
                if nd["op"] == "maxpool":
                    if nd["name"] not in qn._pooled:
                        binding.qmaxpool_i8(qn.bufs[nd["src"]], nd["R"], nd["S"], nd["stride"], nd["pad"],
                                            out=qn.bufs[nd["dst"]])
                else:
                    qn.handles[nd["name"]].run(qn.bufs[nd["src"]], qn._conv_dst(nd), qn._residual(nd))
            b.record()
            torch.cuda.synchronize()
            per[nd["name"]].append(a.elapsed_time(b) / train)
    pk = measured_peaks()
    int8_peak = 2.0 * pk["bf16"]
    print("%-12s %9s %8s %8s %6s  %s" % ("layer", "us", "TOPS", "algGB/s", "roof", "plan"), file=sys.stderr)
    for nd in net["nodes"]:
        ms = float(np.median(per[nd["name"]]))
        if nd["op"] == "maxpool":
            if nd["name"] in qn._pooled:
                print("%-12s %9s  maxpool, taken inside the layer before it" % (nd["name"], "-"), file=sys.stderr)
            else:
                print("%-12s %9.1f  maxpool" % (nd["name"], 1e3 * ms), file=sys.stderr)
            continue
        ops, byt = 2 * wl.conv_macs(nd, N), wl.conv_alg_bytes(nd, N)
        t_ideal = max(ops / (int8_peak * 1e12), byt / (pk["hbm_gbs"] * 1e9)) * 1e3
        print("%-12s %9.1f %8.1f %8.1f %6.3f  %s" % (nd["name"], ms * 1e3, ops / ms / 1e9, byt / ms / 1e6, t_ideal / ms,
                                                     qn.handles[nd["name"]].describe()), file=sys.stderr)


def spawn_ranks(n):
    """`--gpus N` without a launcher: start N ranks of this script, one per GPU, and hand back their exit code."""
    import torch
    if torch.cuda.device_count() < n:
        print("bench.py: --gpus %d but only %d CUDA device(s) visible" % (n, torch.cuda.device_count()), file=sys.stderr)
        return 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--sets", type=int, default=10, help="repetitions of the timed set of --steps replays (median reported)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(WORKLOADS),
                    help="time this stack alone (default: the ResNet-50 headline plus the other configurations)")
    ap.add_argument("--per-layer", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only")
    ap.add_argument("--pool", action="store_true", help="with --layer: take the 2x2 max-pool inside the layer")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--graph-form", default=None, choices=["chain", "branches", "split2"],
                    help="how the step is recorded (default: the fastest of the forms that apply)")
    ap.add_argument("--layer", default=None, help="time one layer of the workload on seeded int8 input")
    ap.add_argument("--batch", type=int, default=None, help="with --layer: batch override")
    ap.add_argument("--single-conv", action="store_true", help="latency of the one-layer configuration")
    ap.add_argument("--calib-elems", type=int, default=0,
                    help="time qcalib_collect alone on this many ReLU-like float32 values")
    ap.add_argument("--mma-peak", action="store_true", help="the tensor pipe's int8 ceiling (MMA-only microbenchmark)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    headline = args.workload or "resnet50"
    make, desc = WORKLOADS[headline]
    if args.impl == "reference":
        return run_reference(args, make(), desc)

    env_world = os.environ.get("WORLD_SIZE")
    if env_world is None and args.gpus > 1:
        sys.exit(spawn_ranks(args.gpus))
    world = int(env_world or "1")
    if world != args.gpus:
        print("bench.py: --gpus %d does not match WORLD_SIZE %d" % (args.gpus, world), file=sys.stderr)
        sys.exit(2)

    import torch
    import torch.distributed as dist
    from paper_1805_07941_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.lib()                                            # fails loudly if the CUDA library is missing
    if args.single_conv:
        return print(json.dumps(single_conv_call(args.warmup, args.steps)))
    if args.calib_elems:
        return print(json.dumps(calib_call(args.calib_elems, args.warmup, args.steps)))
    if args.mma_peak:
        return print(json.dumps(mma_peak_call()))
    if args.layer:
        return run_single_layer(args, make(), desc)

    flush = torch.empty(256 << 20, dtype=torch.int8, device="cuda")
    res, qn, x_host, x_pinned, (net, weights) = measure_network(headline, args, rank, world, flush, True)
    N = net["input"][0]

    # end to end through the public API: pinned host input -> device, run, result -> pinned host
    from paper_1805_07941_b200 import dist as qdist
    out_host = torch.empty(qn.bufs[qn.last].shape, dtype=torch.int8).pin_memory()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if qn.graph is not None:
        # the library's pipelined call: copies of neighbouring steps overlap the layers of this one
        qn.run_pipelined([x_pinned] * args.warmup, [out_host] * args.warmup)
        torch.cuda.synchronize()
        e0.record()
        qn.run_pipelined([x_pinned] * args.steps, [out_host] * args.steps)
        e1.record()
    else:
        for i in range(args.warmup + args.steps):
            if i == args.warmup:
                torch.cuda.synchronize()
                e0.record()
            y = qn.run(x_pinned.cuda(non_blocking=True))
            out_host.copy_(y, non_blocking=True)
        e1.record()
    torch.cuda.synchronize()
    e2e_ms = qdist.max_over_ranks(e0.elapsed_time(e1), device="cuda")
    e2e = {"value": world * N * args.steps / (e2e_ms * 1e-3), "unit": "img/s",
           "h2d_bytes_per_step": int(x_pinned.numel() * 4), "d2h_bytes_per_step": int(out_host.numel())}
    if args.per_layer and rank == 0:
        per_layer_table(qn, net, flush)
    qn.destroy()
    del qn

    extras = None
    if world == 1 and args.workload is None and not args.no_extras:
        extras = {}
        for name in ("vgg16", "inception", "mobilenet"):
            r, _, _, _, _ = measure_network(name, args, rank, world, flush, False)
            extras[name] = r
        extras["single_conv"] = single_conv_call(args.warmup, args.steps)
        extras["calibration"] = calib_call(128 << 20, args.warmup, max(5, args.steps // 3))
        extras["int8_mma_peak"] = mma_peak_call()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_rate(net, weights, x_host)
    if rank == 0:
        pk = measured_peaks()
        print(json.dumps({
            "metric": METRIC, "value": res["img_per_s"], "unit": "img/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "ms_per_step_sets": res["ms_per_step_sets"],
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": desc, "batch_per_gpu": N, "parallelism": "dp%d (replicas, no collective)" % world,
                       "l2": "flushed between timed steps (256 MiB write, untimed)",
                       "timing": "%d sets of %d graph replays, each replay between CUDA events; median set" % (
                           args.sets, args.steps),
                       "graph": res["graph"], "graph_form": res["graph_form"],
                       "graph_forms_tried_ms": res["graph_forms_tried_ms"]},
            "tops": res["tops"], "clocks": res["clocks"], "e2e": e2e,
            "gpu_launches": res["launches_per_step"] * args.steps * args.sets, "roofline": res["roofline"],
            "peaks": {"hbm_gbs": pk["hbm_gbs"], "int8_tops_burst_2x_bf16": 2 * pk["bf16"],
                      "int8_tops_sustained_2x_bf16": 2 * pk["bf16_sustained"], "int8_tops_nominal": NOMINAL_INT8_TOPS,
                      "hbm_gbs_nominal": NOMINAL_HBM_GBS, "source": pk["source"]},
            "calibration_s": res["calibration_s"], "workloads": extras, "cpu_baseline": cpu}))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
