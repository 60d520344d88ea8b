#!/usr/bin/env python3
"""Benchmark of the pattern-pruned 3x3 convolution path.

One step = one pass over all thirteen 3x3 layers of the VGG-16 stack (batch 1
per GPU, fp32, 8-pattern library, 70 % of kernels removed except in the first
layer), each layer on its own seeded synthetic input, packed weights resident
on the device.  The metric is useful GFLOP/s: 2 * 4 * surviving kernels *
output pixels / time, i.e. structural non-zeros only.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Before the timed region the library's own microbenchmarks measure the rates of
the fp32 FMA pipe (scalar and packed) and of the integer dot-product pipe, and
the launch floor of a kernel shaped like the convolution kernels; the roofline
figures are taken against those measured rates.  After the headline workload
the other named workloads (single layer, ResNet-50 and ResNet-18 3x3 stacks,
the large-batch points of the single-layer sweep) are timed the same way and
reported under "configs".

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank
runs the same stack on its own image: images are independent, so there is no
data-path collective; the reported value is the work of all ranks over the
slowest rank's time (weak scaling).  `--impl reference` times the CPU oracle
on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2206_10620_b200 import workloads as wl  # noqa: E402

METRIC = "pattern-pruned conv3x3 useful GFLOP/s (VGG-16 3x3 stack, non-zero MACs only)"
UNIT = "GFLOP/s"
# FP32 pipe peak from unit counts and the maximum SM clock:
# 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz.
FP32_DERIVED_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
KERNEL_SOURCES = ["paper_2206_10620_b200/csrc/patconv.cu", "paper_2206_10620_b200/csrc/gen_core.py",
                  "paper_2206_10620_b200/csrc/pack.cpp"]
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_vgg16_step.txt")


def kernel_source_digest() -> str:
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """DRAM bytes per launch of the convolution kernel from the committed ncu capture, or None
    when the kernel sources have changed since that capture was taken."""
    try:
        txt = open(TRAFFIC_FILE).read()
        dig = re.search(r"kernel_source_digest:\s*(\w+)", txt).group(1)
        val = float(re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", txt).group(1))
    except Exception:
        return None
    return val if dig == kernel_source_digest() else None


def rank_seed(rank: int) -> int:
    """Every rank draws its own image (weak scaling: the batch is sharded by rank)."""
    return wl.BASE_SEED + rank


def max_over_ranks(x: float, dist, device) -> float:
    """The job's time is the slowest rank's (all-reduce MAX; identity for one rank)."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gflops(useful_macs_per_rank: int, world: int, ms: float) -> float:
    """Useful GFLOP/s of all ranks together over the slowest rank's time."""
    return 2.0 * useful_macs_per_rank * world / (ms * 1e-3) / 1e9


def workload(name="vgg16"):
    return wl.CONFIGS[name]()


def measured_hbm_gbs():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"], "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            time.sleep(0.1)                      # the first sample is there before the region starts
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def oracle_sample(specs, budget_s=15.0):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: whole layers,
    smallest first, as many as fit the time budget; when the whole stack fits several times
    over, whole passes are repeated until about two thirds of the budget are used."""
    import oracle
    order = sorted(range(len(specs)), key=lambda i: specs[i].dense_macs())
    t_total, macs, dense, used, rate, passes = 0.0, 0, 0, [], None, 0
    data = {}
    while True:
        took_all = True
        for i in order:
            s = specs[i]
            if rate is not None and t_total + s.dense_macs() / rate > budget_s:
                took_all = False
                continue
            if i not in data:
                data[i] = wl.make_layer(s)
            d = data[i]
            t0 = time.perf_counter()
            oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=s.relu, stride=s.stride)
            dt = time.perf_counter() - t0
            t_total += dt
            macs += s.useful_macs()
            dense += s.dense_macs()
            if passes == 0:
                used.append(s.name)
            rate = dense / t_total
        passes += 1
        if not took_all or t_total > 0.66 * budget_s or t_total * (passes + 1) / passes > budget_s:
            break
    return {"value": 2.0 * macs / t_total / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "whole layers %s of the stack, %d pass(es) (%.2f dense GMAC; the stack has %.2f), %.1f s" % (
                ",".join(used), passes, dense / 1e9, sum(s.dense_macs() for s in specs) / 1e9, t_total),
            "seconds": t_total}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    specs = workload()
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(specs, budget_s=per_step)
        if i >= args.warmup:
            vals.append(r)
    v = float(np.mean([r["value"] for r in vals]))
    ms = float(np.mean([r["seconds"] for r in vals])) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "vgg16 3x3 stack, batch 1, fp32, 8 patterns, 70% kernels removed; "
                                   "each step a bounded sample of whole layers"},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class Stack:
    """The layers of one workload on the device: packed, planned, with inputs and outputs."""

    def __init__(self, specs, seed, device_index, plan=True, keep_host=True, no_small_blocks=False):
        import torch
        from paper_2206_10620_b200 import binding
        self.torch = torch
        self.specs = specs
        dev = torch.device("cuda", device_index)
        tdt = {"f32": torch.float32, "f16": torch.float16, "i8": torch.int32}
        self.layers = []
        for s in specs:
            d = wl.make_layer(s, seed=seed)
            pk = binding.Packed(s.c_in, s.c_out, s.stride, s.dtype, d.masks, d.w, d.pid, device=device_index)
            if plan:
                pk.plan(s.n, s.h, s.w, no_small_blocks=no_small_blocks)
            x = torch.from_numpy(d.x).to(dev)
            b = torch.from_numpy(d.bias).to(dev)
            y = torch.empty((s.n, s.ho, s.wo, s.c_out), dtype=tdt[s.dtype], device=dev)
            if not keep_host:
                d.x = None
            self.layers.append((s, d, pk, x, b, y))
        self.useful = sum(s.useful_macs() for s in specs)
        self.dense = sum(s.dense_macs() for s in specs)

    def step(self, stream):
        for (s, d, pk, x, b, y) in self.layers:
            pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), s.relu, y.data_ptr(), stream)

    def timed_steps(self, stream, steps, flush):
        """`steps` passes, each bracketed by CUDA events on the launching stream; with `flush`, a
        write of more than the L2's size between the steps (outside the event pairs)."""
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for k in range(steps):
            if flush is not None:
                flush.fill_(k & 0xFF)
            ev[k][0].record()
            self.step(stream)
            ev[k][1].record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]


def stats(ms_list):
    a = np.asarray(ms_list, dtype=np.float64)
    return {"mean": float(a.mean()), "median": float(np.median(a)), "min": float(a.min()), "max": float(a.max())}


def layer_bounds(s, fp32_tflops, dp4a_tmacs, hbm_gbs):
    """Ideal times of one layer in seconds: on the fp32 FMA pipe (what every variant runs on), on
    the integer dot-product pipe (the int8 variant's other yardstick) and on HBM."""
    t_fp32 = 2.0 * s.useful_macs() / (fp32_tflops * 1e12)
    t_dp4a = s.useful_macs() / (dp4a_tmacs * 1e12) if s.dtype == "i8" else None
    t_hbm = s.compulsory_bytes() / (hbm_gbs * 1e9)
    return t_fp32, t_dp4a, t_hbm


def time_block_gemm(torch, binding, dev, stream, flush, fp32_tflops, hbm_gbs, oracle_check=True, only="", reps=5):
    """Times xgen_blockgemm_run on the 1x1 layers of ResNet-50 in matrix form.  Per layer: median
    microseconds, useful TFLOP/s (kept weights only), the fraction of the fp32 FMA pipe and of the
    binding roofline (the slower of kept multiply-adds on that pipe and compulsory bytes at HBM rate)."""
    out = {"layers": [], "recipe": "ResNet-50 1x1 convolutions as [batch*pixels, c_in] x [c_out, c_in]^T, batch 32, fp16 storage, "
                                   "32x32 pruning blocks, 40 % of rows and 40 % of columns kept per block"}
    t_all = ideal_all = flops_all = 0.0
    for spec in wl.config_resnet50_1x1():
        if only and not spec.name.startswith(only):
            continue
        d = wl.make_block_gemm(spec)
        pk = binding.BlockGemm(spec.k, spec.c_out, spec.br, spec.bc, spec.dtype, d.w, d.row_keep, d.col_keep, device=dev.index)
        x = torch.from_numpy(d.x).to(dev)
        b = torch.from_numpy(d.bias).to(dev)
        y = torch.empty((spec.m, spec.c_out), dtype=x.dtype, device=dev)
        for _ in range(3):
            pk.run(x.data_ptr(), spec.m, b.data_ptr(), True, y.data_ptr(), stream)
        torch.cuda.synchronize()
        ts = []
        for r in range(reps):
            flush.fill_(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            pk.run(x.data_ptr(), spec.m, b.data_ptr(), True, y.data_ptr(), stream)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        us = float(np.median(ts)) * 1e3
        macs = d.useful_macs()
        t_alu = 2.0 * macs / (fp32_tflops * 1e12)
        t_hbm = d.compulsory_bytes() / (hbm_gbs * 1e9)
        rec = {"layer": spec.name, "rows": spec.m, "us": round(us, 2), "useful_tflops": round(2.0 * macs / us * 1e-6, 2),
               "dense_equiv_tflops": round(2.0 * d.dense_macs() / us * 1e-6, 2),
               "frac_of_fp32_pipe": round(t_alu * 1e6 / us, 4), "bound": "alu" if t_alu >= t_hbm else "hbm",
               "ideal_us": round(max(t_alu, t_hbm) * 1e6, 2), "frac_of_binding_roofline": round(max(t_alu, t_hbm) * 1e6 / us, 4)}
        if oracle_check and spec.m <= 8192:
            import oracle
            got = y[:256].cpu().numpy().astype(np.float64)
            ref, S = oracle.block_gemm(d.x[:256], d.w, d.row_keep, d.col_keep, spec.br, spec.bc, bias=d.bias, relu=True, with_scale=True)
            rec["parity_ok"] = bool((np.abs(got - ref) <= 2e-3 * np.maximum(np.abs(ref), 0.01 * S) + 1e-30).all())
        out["layers"].append(rec)
        t_all += us
        ideal_all += max(t_alu, t_hbm) * 1e6
        flops_all += 2.0 * macs
        del pk, x, b, y
    torch.cuda.empty_cache()
    if t_all > 0:
        out["total_us"] = round(t_all, 1)
        out["useful_tflops"] = round(flops_all / t_all * 1e-6, 2)
        out["frac_of_fp32_pipe"] = round(flops_all / t_all * 1e-6 / fp32_tflops, 4)
        out["frac_of_binding_roofline"] = round(ideal_all / t_all, 4)
    return out


def time_depthwise(torch, binding, dev, stream, flush, hbm_gbs, oracle_check=True, only="", reps=5):
    """Times xgen_dwconv_run on the depthwise 3x3 layers of a MobileNet-v1-shaped network (batch 32,
    fp16 storage).  The layer is bound by HBM: per layer the achieved rate of its compulsory bytes
    (x once, y once, kept weights) and that rate's fraction of the measured copy rate."""
    out = {"layers": [], "recipe": "depthwise 3x3 layers of a MobileNet-v1-shaped network, batch 32, fp16 storage, NHWC, "
                                   "8-pattern library, bias+ReLU fused"}
    t_all = b_all = 0.0
    for spec in wl.config_mobilenet_depthwise():
        if only and not spec.name.startswith(only):
            continue
        d = wl.make_depthwise(spec)
        pk = binding.Depthwise(spec.c, spec.stride, spec.dtype, d.masks, d.w, d.pid, device=dev.index)
        x = torch.from_numpy(d.x).to(dev)
        b = torch.from_numpy(d.bias).to(dev)
        y = torch.empty((spec.n, spec.ho, spec.wo, spec.c), dtype=x.dtype, device=dev)
        for _ in range(3):
            pk.run(x.data_ptr(), spec.n, spec.h, spec.w, b.data_ptr(), True, y.data_ptr(), stream)
        torch.cuda.synchronize()
        ts = []
        for r in range(reps):
            flush.fill_(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            pk.run(x.data_ptr(), spec.n, spec.h, spec.w, b.data_ptr(), True, y.data_ptr(), stream)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        us = float(np.median(ts)) * 1e3
        nbytes = spec.compulsory_bytes()
        rec = {"layer": spec.name, "us": round(us, 2), "mbytes": round(nbytes / 1e6, 1), "gbs": round(nbytes / us * 1e-3, 1),
               "frac_of_hbm": round(nbytes / us * 1e-3 / hbm_gbs, 4), "useful_gflops": round(2.0 * spec.useful_macs() / us * 1e-3, 1)}
        if oracle_check and spec.c >= 512:
            import oracle
            got = y[:1].cpu().numpy().astype(np.float64)
            ref, S = oracle.depthwise(d.x[:1], d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=spec.stride, with_scale=True)
            rec["parity_ok"] = bool((np.abs(got - ref) <= 2e-3 * np.maximum(np.abs(ref), 0.01 * S) + 2.0 ** -25).all())
        out["layers"].append(rec)
        t_all += us
        b_all += nbytes
        del pk, x, b, y
    torch.cuda.empty_cache()
    if t_all > 0:
        out["total_us"] = round(t_all, 1)
        out["gbs"] = round(b_all / t_all * 1e-3, 1)
        out["frac_of_hbm"] = round(b_all / t_all * 1e-3 / hbm_gbs, 4)
    return out


def run_gpu(args):
    import torch
    from paper_2206_10620_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    binding.lib()                                   # fail loudly if the CUDA library is missing

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # --- pipe rates and launch floor, measured in this process before anything is timed
    probe = binding.probe(local)
    fp32_peak = max(probe["ffma_tflops"], probe["ffma2_tflops"])
    dp4a_peak = probe["dp4a_tmacs"]
    hbm, hbm_src = measured_hbm_gbs()

    if args.block_gemm_only:                        # profiling aid: one layer of the matrix products, nothing else
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        rec = time_block_gemm(torch, binding, dev, torch.cuda.current_stream().cuda_stream, flush, fp32_peak, hbm,
                              oracle_check=False, only=args.block_gemm_only, reps=3)
        print(json.dumps({"block_gemm": rec, "measured_peaks": probe}), flush=True)
        return

    if args.depthwise_only:                         # profiling aid: one depthwise layer, nothing else
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        rec = time_depthwise(torch, binding, dev, torch.cuda.current_stream().cuda_stream, flush, hbm,
                             oracle_check=False, only=args.depthwise_only, reps=3)
        print(json.dumps({"depthwise": rec}), flush=True)
        return

    specs = workload(args.workload)
    if args.only:
        keep = set(args.only.split(","))
        specs = [s for s in specs if s.name in keep]
    stack = Stack(specs, rank_seed(rank), local)
    stream = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)    # > 126 MB of L2
    warmup = max(3, args.warmup)
    for _ in range(warmup):
        stack.step(stream)
    barrier()

    # --- timed region: K steps, each bracketed by CUDA events, L2 flushed between steps
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.launch_count()
    barrier()
    ms_steps = stack.timed_steps(stream, args.steps, flush)
    barrier()
    launches = binding.launch_count() - launches0
    # The K steps above are the reported value.  The same protocol then runs on, outside that
    # value, until at least `--stat-steps` steps have been timed: median and minimum of a
    # region long enough for the clock sampler to see it.
    extra = stack.timed_steps(stream, max(0, args.stat_steps - args.steps), flush) if args.stat_steps > args.steps else []
    clocks = sampler.stop()
    st_flushed = stats(ms_steps)
    st_long = stats(ms_steps + extra)
    st_long["steps"] = len(ms_steps) + len(extra)
    ms = max_over_ranks(st_flushed["mean"], dist, dev)
    useful, dense = stack.useful, stack.dense
    value = whole_job_gflops(useful, world, ms)
    # the same steps with whatever the previous step left in L2 (no flush)
    st_warm = stats(stack.timed_steps(stream, max(args.steps, 50), None))

    # --- per-layer device times (L2 flushed before each layer) beside each layer's ideal times
    per_layer = []
    for (s, d, pk, x, b, y) in stack.layers:
        ts = []
        for r in range(7):
            flush.fill_(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), s.relu, y.data_ptr(), stream)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        t_ms = float(np.median(ts))
        t_fp32, t_dp4a, t_hbm = layer_bounds(s, fp32_peak, dp4a_peak, hbm)
        info = pk.plan_info(s.n, s.h, s.w)
        rec = {"layer": s.name, "us": round(t_ms * 1e3, 2), "us_min": round(min(ts) * 1e3, 2),
               "ideal_us": round(max(t_fp32, t_hbm) * 1e6, 2), "launch_floor_us": round(probe["launch_floor_us"], 2),
               "useful_gflops": round(2.0 * s.useful_macs() / t_ms / 1e6, 1),
               "dense_equiv_gflops": round(2.0 * s.dense_macs() / t_ms / 1e6, 1),
               "bound": "alu" if t_fp32 >= t_hbm else "hbm",
               "roofline_frac": round(max(t_fp32, t_hbm) / (t_ms * 1e-3), 4),
               "grid": "%d tiles x %d filter blocks x %d splits" % (info["tiles"], info["filter_blocks"], info["splits"])}
        if t_dp4a is not None:
            rec["roofline_frac_dp4a"] = round(max(t_dp4a, t_hbm) / (t_ms * 1e-3), 4)
        per_layer.append(rec)
    layer_ms = sum(p["us"] for p in per_layer) * 1e-3

    # The dominant kernel is the only kernel of the step: its achieved rate is the step's useful
    # flops over the timed region (this rank's K steps, events on the launching stream).
    own_ms = st_flushed["mean"]
    achieved = 2.0 * useful / (own_ms * 1e-3) / 1e12
    binding_ms = sum(max(layer_bounds(s, fp32_peak, dp4a_peak, hbm)[0], layer_bounds(s, fp32_peak, dp4a_peak, hbm)[2])
                     for s in specs) * 1e3
    med_mhz = clocks.get("sm_mhz") or 0.0
    roofline = {"bound": "alu", "achieved": achieved, "peak": fp32_peak, "unit": "TFLOP/s",
                "frac": achieved / fp32_peak,
                "traffic": recorded_traffic() if args.workload == "vgg16" and not args.only else None,
                "kernel": "patconv_kernel (all %d layers of the step)" % len(specs),
                "peak_source": "measured in this run: register-only fp32 FMA microbenchmarks at full occupancy "
                               "(scalar %.1f, packed %.1f TFLOP/s); derived 148 SMs x 128 lanes x 2 x 1.965 GHz = %.2f"
                               % (probe["ffma_tflops"], probe["ffma2_tflops"], FP32_DERIVED_TFLOPS),
                "peak_derived": FP32_DERIVED_TFLOPS, "frac_of_derived_peak": achieved / FP32_DERIVED_TFLOPS,
                "hbm_peak_gbs": hbm, "hbm_peak_source": hbm_src,
                "binding_roofline_ms": binding_ms, "frac_of_binding_roofline": binding_ms / own_ms,
                "isolated_layers_ms": layer_ms,
                "frac_isolated_layers": 2.0 * useful / (layer_ms * 1e-3) / 1e12 / fp32_peak,
                "ms_x_median_sm_mhz": own_ms * med_mhz,
                "frac_at_sampled_clock": (achieved / (fp32_peak * med_mhz / probe["sm_clock_mhz"])
                                          if med_mhz and probe["sm_clock_mhz"] else None)}

    # --- parity of what was timed: the three smallest layers against the CPU oracle (outside the timing)
    parity_checked = []
    if rank == 0 and not args.no_parity:
        import oracle
        for (s, d, pk, x, b, y) in sorted(stack.layers, key=lambda t: t[0].dense_macs())[:3]:
            got = y.cpu().numpy()
            if s.dtype == "i8":
                ref = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=s.relu, stride=s.stride)
                ok = bool(np.array_equal(got.astype(np.int64), ref))
            else:
                ref, S = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=s.relu, stride=s.stride, with_scale=True)
                tol = 1e-4 if s.dtype == "f32" else 2e-3
                ok = bool((np.abs(got.astype(np.float64) - ref) <= tol * np.maximum(np.abs(ref), 0.01 * S) + 1e-30).all())
            parity_checked.append({"layer": s.name, "ok": ok})
            if not ok:
                raise SystemExit("bench: layer %s does not match the oracle" % s.name)

    # --- host cost of one xgen_patconv_run call on a prepared handle
    (s, d, pk, x, b, y) = min(stack.layers, key=lambda t: t[0].useful_macs())
    torch.cuda.synchronize()
    n_calls = 500
    t0 = time.perf_counter()
    for _ in range(n_calls):
        pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), s.relu, y.data_ptr(), stream)
    host_us = (time.perf_counter() - t0) / n_calls * 1e6
    torch.cuda.synchronize()

    # --- end to end through the host-buffer entry point (xgen_patconv_enqueue_host; copies inside the timed
    # region): inputs and results live in pinned host memory; every step copies every layer's input and bias
    # to the device and its result back.
    e2e_steps = max(1, min(args.steps, 5))
    pinned = []
    for (s, d, pk, x, b, y) in stack.layers:
        hx = torch.from_numpy(d.x).pin_memory()
        hb = torch.from_numpy(d.bias).pin_memory()
        hy = torch.empty(y.shape, dtype=y.dtype).pin_memory()
        pinned.append((hx, hb, hy))
    h2d = sum(hx.numel() * hx.element_size() + hb.numel() * hb.element_size() for hx, hb, hy in pinned)
    d2h = sum(hy.numel() * hy.element_size() for hx, hb, hy in pinned)

    def e2e_step():
        # every layer is enqueued (copy in, kernel, copy out) without waiting; the copies of one
        # layer overlap the kernels and the opposite copies of its neighbours; then wait for all
        for (s, d, pk, x, b, y), (hx, hb, hy) in zip(stack.layers, pinned):
            pk.enqueue_host_ptr(hx.data_ptr(), s.n, s.h, s.w, hb.data_ptr(), s.relu, hy.data_ptr(), stream)
        for (s, d, pk, x, b, y) in stack.layers:
            pk.sync(stream)

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, dist, dev)
    e2e = {"value": 2.0 * useful * world / e2e_s / 1e9, "unit": UNIT,
           "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_s * 1e3}

    # --- the other named workloads, timed the same way (fewer steps), one after the other
    configs = {}
    if rank == 0 and world == 1 and not args.no_configs and args.workload == "vgg16" and not args.only:
        del pinned
        others = [("single", wl.config_single_layer()), ("resnet50", wl.config_resnet50()),
                  ("resnet18", wl.config_resnet18())]
        sweep = {s.name: s for s in wl.config_sweep()}
        for p in ("0.0", "0.5", "0.75", "0.875"):
            others.append(("sweep_n256_p%s" % p, [sweep["sweep_n256_p%s_lib8" % p]]))
        for name, sp in others:
            stk = Stack(sp, wl.BASE_SEED, local, keep_host=False)
            for _ in range(3):
                stk.step(stream)
            torch.cuda.synchronize()
            st_c = stats(stk.timed_steps(stream, args.config_steps, flush))
            t = st_c["median"] * 1e-3
            bind = sum(max(layer_bounds(s, fp32_peak, dp4a_peak, hbm)[0], layer_bounds(s, fp32_peak, dp4a_peak, hbm)[2])
                       for s in sp)
            rec = {"ms_per_step": st_c, "steps": args.config_steps, "layers": len(sp), "dtype": sp[0].dtype,
                   "batch": sp[0].n, "useful_tflops": 2.0 * stk.useful / t / 1e12,
                   "dense_equiv_tflops": 2.0 * stk.dense / t / 1e12,
                   "frac_of_fp32_pipe": 2.0 * stk.useful / t / 1e12 / fp32_peak,
                   "binding_roofline_ms": bind * 1e3, "frac_of_binding_roofline": bind / t}
            if sp[0].dtype == "i8":
                bind_d = sum(max(layer_bounds(s, fp32_peak, dp4a_peak, hbm)[1], layer_bounds(s, fp32_peak, dp4a_peak, hbm)[2])
                             for s in sp)
                rec["frac_of_dp4a_pipe"] = stk.useful / t / 1e12 / dp4a_peak
                rec["frac_of_binding_roofline_dp4a"] = bind_d / t
            configs[name] = rec
            del stk
            torch.cuda.empty_cache()

    # --- operators fused behind the convolution: what they save on the layers that feed a pooling
    # (VGG-16's stage ends) and on the integer stack (uint8 codes instead of int32 sums)
    fused = {}
    if rank == 0 and world == 1 and not args.no_configs and args.workload == "vgg16" and not args.only:
        def time_layers(stk, runner, reps=7):
            out = []
            for item in stk.layers:
                ts = []
                for r in range(reps):
                    flush.fill_(r)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    runner(item)
                    e1.record()
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1))
                out.append(float(np.median(ts)) * 1e3)
            return out

        ends = [s for s in wl.config_vgg16() if s.name in ("conv2", "conv4", "conv7", "conv10", "conv13")]
        stk = Stack(ends, wl.BASE_SEED, local, keep_host=False, no_small_blocks=True)   # the fused operators need 4x4 blocks
        plain_us = time_layers(stk, lambda it: it[2].run(it[3].data_ptr(), it[0].n, it[0].h, it[0].w, it[4].data_ptr(),
                                                         True, it[5].data_ptr(), stream))
        pooled = [torch.empty((s.n, s.ho // 2, s.wo // 2, s.c_out), dtype=torch.float32, device=dev) for s in ends]
        pool_us = time_layers(stk, lambda it: it[2].run_fused(it[3].data_ptr(), it[0].n, it[0].h, it[0].w, it[4].data_ptr(),
                                                              pooled[ends.index(it[0])].data_ptr(), stream, relu=True, pool=2))
        fused["vgg16_stage_ends_maxpool"] = {
            "layers": [s.name for s in ends], "plain_us": [round(t, 2) for t in plain_us],
            "fused_pool_us": [round(t, 2) for t in pool_us],
            "result_bytes_plain": int(sum(s.n * s.ho * s.wo * s.c_out * 4 for s in ends)),
            "result_bytes_fused": int(sum(s.n * s.ho * s.wo * s.c_out for s in ends)),
            "note": "the unfused network also reads the full result back and writes the pooled one"}
        del stk, pooled
        sp = wl.config_resnet18()
        stk = Stack(sp, wl.BASE_SEED, local, keep_host=False)
        plain_us = time_layers(stk, lambda it: it[2].run(it[3].data_ptr(), it[0].n, it[0].h, it[0].w, it[4].data_ptr(),
                                                         True, it[5].data_ptr(), stream), reps=5)
        codes = [torch.empty((s.n, s.ho, s.wo, s.c_out), dtype=torch.uint8, device=dev) for s in sp]
        scales = [torch.full((s.c_out,), 1e-3, dtype=torch.float32, device=dev) for s in sp]
        rq_us = time_layers(stk, lambda it: it[2].run_fused(it[3].data_ptr(), it[0].n, it[0].h, it[0].w, it[4].data_ptr(),
                                                            codes[sp.index(it[0])].data_ptr(), stream, relu=True,
                                                            requant_scale_ptr=scales[sp.index(it[0])].data_ptr()), reps=5)
        fused["resnet18_requantised"] = {
            "plain_int32_ms": round(sum(plain_us) * 1e-3, 4), "fused_uint8_ms": round(sum(rq_us) * 1e-3, 4),
            "result_bytes_plain": int(sum(s.n * s.ho * s.wo * s.c_out * 4 for s in sp)),
            "result_bytes_fused": int(sum(s.n * s.ho * s.wo * s.c_out for s in sp))}
        del stk, codes, scales
        torch.cuda.empty_cache()

    # --- the block-pruned matrix product on ResNet-50's 1x1 convolutions (batch 32, fp16 storage,
    # 32 x 32 blocks keeping 40 % of their rows and 40 % of their columns: about one sixth of the
    # weights), each layer alone after an L2 flush
    block_gemm = {}
    if rank == 0 and world == 1 and not args.no_configs and args.workload == "vgg16" and not args.only:
        block_gemm = time_block_gemm(torch, binding, dev, stream, flush, fp32_peak, hbm, oracle_check=not args.no_parity)

    depthwise = {}
    if rank == 0 and world == 1 and not args.no_configs and args.workload == "vgg16" and not args.only:
        depthwise = time_depthwise(torch, binding, dev, stream, flush, hbm, oracle_check=not args.no_parity)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = oracle_sample(specs, budget_s=args.cpu_seconds)
        cpu.pop("seconds", None)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": "vgg16 3x3 stack (13 layers, 224..14 px), batch 1 per GPU, fp32, NHWC, "
                                       "8-pattern library, 70% of kernels removed (0% in layer 1), bias+ReLU fused"
                           if args.workload == "vgg16" else args.workload,
                           "l2": "flushed between timed steps (256 MB write)",
                           "useful_gmac_per_step": useful / 1e9, "dense_gmac_per_step": dense / 1e9},
                "ms_per_step_stats": st_flushed, "ms_per_step_stats_long": st_long, "ms_per_step_l2_warm": st_warm,
                "dense_equiv_gflops": 2.0 * dense * world / (ms * 1e-3) / 1e9,
                "net_ms_per_batch": ms,
                "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e,
                "roofline": roofline, "measured_peaks": probe, "host_us_per_run_call": round(host_us, 2),
                "parity_checked": parity_checked, "cpu_baseline": cpu, "per_layer": per_layer, "configs": configs, "fused": fused,
                "block_gemm": block_gemm, "depthwise": depthwise}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--stat-steps", type=int, default=300,
                    help="keep timing steps, outside the reported value, until this many are in the statistics")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg16", choices=list(wl.CONFIGS))
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--config-steps", type=int, default=10, help="timed steps of each of the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-configs", action="store_true", help="skip the other named workloads")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle comparison of the timed layers")
    ap.add_argument("--block-gemm-only", default="", help="time only this layer of the block-pruned matrix products "
                    "(a prefix of its name, e.g. pw5) and print its record: profiling aid")
    ap.add_argument("--depthwise-only", default="", help="time only this depthwise layer (a prefix of its name, e.g. dw3): "
                    "profiling aid")
    ap.add_argument("--only", default="", help="comma-separated layer names: restrict the stack (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
