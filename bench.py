#!/usr/bin/env python3
"""Benchmark of the pattern-pruned 3x3 convolution path.

One step = one pass over all thirteen 3x3 layers of the VGG-16 stack (batch 1
per GPU, fp32, 8-pattern library, 70 % of kernels removed except in the first
layer), each layer on its own seeded synthetic input, packed weights resident
on the device.  The metric is useful GFLOP/s: 2 * 4 * surviving kernels *
output pixels / time, i.e. structural non-zeros only.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank
runs the same stack on its own image: images are independent, so there is no
data-path collective; the reported value is the work of all ranks over the
slowest rank's time (weak scaling).  `--impl reference` times the CPU oracle
on the host cores instead (rank 0 only).
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

from paper_2206_10620_b200 import workloads as wl  # noqa: E402

METRIC = "pattern-pruned conv3x3 useful GFLOP/s (VGG-16 3x3 stack, non-zero MACs only)"
UNIT = "GFLOP/s"
# FP32 pipe peak from unit counts and the maximum SM clock:
# 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz.
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


# dram__bytes_read.sum + dram__bytes_write.sum of patconv_kernel, average per launch over one
# step of this workload, from the ncu capture summarised in profiles/bench_vgg16_launch_list.md
# (taken with the kernels as committed; set to None when the kernel changes).
NCU_DRAM_BYTES_PER_LAUNCH = 5.6e6


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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
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
    """Time the CPU oracle, as it stands, on a bounded sample of the workload:
    whole layers, smallest first, until the time budget is used."""
    import oracle
    order = sorted(range(len(specs)), key=lambda i: specs[i].dense_macs())
    t_total, macs, dense, used, rate = 0.0, 0, 0, [], None
    for i in order:
        s = specs[i]
        if rate is not None and t_total + s.dense_macs() / rate > budget_s:
            continue
        d = wl.make_layer(s)
        t0 = time.perf_counter()
        oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=s.relu, stride=s.stride)
        dt = time.perf_counter() - t0
        t_total += dt
        macs += s.useful_macs()
        dense += s.dense_macs()
        used.append(s.name)
        rate = dense / t_total
    return {"value": 2.0 * macs / t_total / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "whole layers %s of the stack (%.2f of %.2f dense GMAC), %.1f s" % (
                ",".join(used), dense / 1e9, sum(s.dense_macs() for s in specs) / 1e9, t_total),
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

    specs = workload(args.workload)
    if args.only:
        keep = set(args.only.split(","))
        specs = [s for s in specs if s.name in keep]
    layers = []
    tdt = {"f32": torch.float32, "f16": torch.float16, "i8": torch.int32}
    for s in specs:
        d = wl.make_layer(s, seed=rank_seed(rank))
        pk = binding.Packed(s.c_in, s.c_out, s.stride, s.dtype, d.masks, d.w, d.pid, device=local)
        pk.plan(s.n, s.h, s.w)
        x = torch.from_numpy(d.x).to(dev)
        b = torch.from_numpy(d.bias).to(dev)
        y = torch.empty((s.n, s.ho, s.wo, s.c_out), dtype=tdt[s.dtype], device=dev)
        layers.append((s, d, pk, x, b, y))
    stream = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)    # > 126 MB of L2

    def step():
        for (s, d, pk, x, b, y) in layers:
            pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), s.relu, y.data_ptr(), stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()

    # --- timed region: K steps, each bracketed by CUDA events, L2 flushed between steps
    sampler = ClockSampler(local)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = binding.launch_count()
    barrier()
    for k in range(args.steps):
        flush.fill_(k & 0xFF)
        ev[k][0].record()
        step()
        ev[k][1].record()
    barrier()
    launches = binding.launch_count() - launches0
    clocks = sampler.stop()
    ms_steps = [a.elapsed_time(b) for a, b in ev]
    ms = max_over_ranks(float(np.mean(ms_steps)), dist, dev)
    useful = sum(s.useful_macs() for s in specs)
    dense = sum(s.dense_macs() for s in specs)
    value = whole_job_gflops(useful, world, ms)

    # --- per-layer device times (L2 flushed before each layer) for the roofline
    hbm, hbm_src = measured_hbm_gbs()
    per_layer = []
    reps = 5
    for (s, d, pk, x, b, y) in layers:
        ts = []
        for r in range(reps):
            flush.fill_(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), s.relu, y.data_ptr(), stream)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        t_ms = float(np.median(ts))
        t_alu = 2.0 * s.useful_macs() / (FP32_PEAK_TFLOPS * 1e12)
        t_hbm = s.compulsory_bytes() / (hbm * 1e9)
        per_layer.append({"layer": s.name, "ms": round(t_ms, 5),
                          "useful_gflops": round(2.0 * s.useful_macs() / t_ms / 1e6, 1),
                          "dense_equiv_gflops": round(2.0 * s.dense_macs() / t_ms / 1e6, 1),
                          "bound": "alu" if t_alu >= t_hbm else "hbm",
                          "roofline_frac": round(max(t_alu, t_hbm) / (t_ms * 1e-3), 4)})
    layer_ms = sum(p["ms"] for p in per_layer)
    # The dominant kernel is the only kernel of the step: its achieved rate is the step's useful
    # flops over the timed region (this rank's K steps, events on the launching stream).  The
    # per-layer times above are taken one launch at a time (nothing overlaps the launch) and are
    # reported beside it.
    own_ms = float(np.mean(ms_steps))
    achieved = 2.0 * useful / (own_ms * 1e-3) / 1e12
    roofline = {"bound": "alu", "achieved": achieved, "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s",
                "frac": achieved / FP32_PEAK_TFLOPS,
                "traffic": NCU_DRAM_BYTES_PER_LAUNCH if args.workload == "vgg16" and not args.only else None,
                "kernel": "patconv_kernel<f32, stride 1, 8 patterns> (all 13 layers)",
                "peak_source": "148 SMs x 128 lanes x 2 x 1.965 GHz (FP32 FMA pipe; derived, not in the measured-peaks file)",
                "hbm_peak_gbs": hbm, "hbm_peak_source": hbm_src,
                "binding_roofline_ms": sum(max(2.0 * s.useful_macs() / (FP32_PEAK_TFLOPS * 1e12),
                                               s.compulsory_bytes() / (hbm * 1e9)) for s in specs) * 1e3,
                "frac_of_binding_roofline": None}
    roofline["frac_of_binding_roofline"] = roofline["binding_roofline_ms"] / own_ms
    roofline["isolated_layers_ms"] = layer_ms
    roofline["frac_isolated_layers"] = 2.0 * useful / (layer_ms * 1e-3) / 1e12 / FP32_PEAK_TFLOPS

    # --- end to end through the host-buffer entry point (xgen_patconv_enqueue_host; copies inside the timed region):
    # inputs and results live in pinned host memory; every step copies every layer's input
    # and bias to the device and its result back.
    e2e_steps = max(1, min(args.steps, 5))
    pinned = []
    for (s, d, pk, x, b, y) in layers:
        hx = torch.from_numpy(d.x).pin_memory()
        hb = torch.from_numpy(d.bias).pin_memory()
        hy = torch.empty(y.shape, dtype=y.dtype).pin_memory()
        pinned.append((hx, hb, hy))
    h2d = sum(hx.numel() * hx.element_size() + hb.numel() * hb.element_size() for hx, hb, hy in pinned)
    d2h = sum(hy.numel() * hy.element_size() for hx, hb, hy in pinned)

    def e2e_step():
        # every layer is enqueued (copy in, kernel, copy out) without waiting; the copies of one
        # layer overlap the kernels and the opposite copies of its neighbours; then wait for all
        st = torch.cuda.current_stream().cuda_stream
        for (s, d, pk, x, b, y), (hx, hb, hy) in zip(layers, pinned):
            pk.enqueue_host_ptr(hx.data_ptr(), s.n, s.h, s.w, hb.data_ptr(), s.relu, hy.data_ptr(), st)
        for (s, d, pk, x, b, y) in layers:
            pk.sync(st)

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

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = oracle_sample(specs, budget_s=args.cpu_seconds)
        cpu.pop("seconds", None)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": "vgg16 3x3 stack (13 layers, 224..14 px), batch 1 per GPU, fp32, NHWC, "
                                       "8-pattern library, 70% of kernels removed (0% in layer 1), bias+ReLU fused",
                           "l2": "flushed between timed steps (256 MB write)",
                           "useful_gmac_per_step": useful / 1e9, "dense_gmac_per_step": dense / 1e9},
                "dense_equiv_gflops": 2.0 * dense * world / (ms * 1e-3) / 1e9,
                "net_ms_per_batch": ms,
                "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e,
                "roofline": roofline, "cpu_baseline": cpu, "per_layer": per_layer}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg16", choices=list(wl.CONFIGS))
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--only", default="", help="comma-separated layer names: restrict the stack (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
