#!/usr/bin/env python
"""Benchmark of the 2:4 sparse convolution forward on B200.

A step is one pass of the masked-convolution forward over every layer of the ResNet-18-shaped
3x3 sweep at batch 32 (seeded synthetic activations and weights, masks by magnitude selected
and compressed once beforehand with the library's own kernels).  The reported value is
dense-equivalent TFLOP/s (2*P*C_out*K per layer) over all ranks.  Each rank rotates over
several input/output buffer sets whose total footprint exceeds the L2 cache, so every step
reads its activations from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dense-equiv TFLOP/s of 2:4 sparse conv fwd (bf16), % of sparse-TC roofline, xdense"
WORKLOADS = {2: "resnet18_3x3_sweep_bf16_nhwc_batch32", 3: "resnet50_bottleneck_layers_bf16_nhwc_batch64",
             4: "convnext_t_pointwise_layers_bf16_nhwc_batch128",
           5: "resnet50_conv_stack_end_to_end_bf16_nhwc_batch256"}
CONFIG_ID = 2          # the benchmarked workload; --workload-config picks another for layer tables
WORKLOAD = WORKLOADS[CONFIG_ID]
L2_BYTES = 126 * 2 ** 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return {"hbm_gbs": float(pk["hbm_gbs"]), "bf16_tflops": float(pk["bf16_tflops"]),
                "bf16_tflops_sustained": float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def timed_layers():
    from paper_2411_00288_b200 import synth
    return [s for s in synth.config_layers(CONFIG_ID) if not s.extra]


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_leg(target_seconds: float = 15.0):
    """Time the fp64 CPU oracle, as it stands, on a bounded sample of the same workload."""
    import numpy as np  # noqa: F401
    from oracle import masks
    from oracle.conv import conv2d_f64, threads
    from paper_2411_00288_b200 import synth
    from tests import parity
    import dataclasses

    def run(batch):
        flops, secs = 0, 0.0
        for spec in timed_layers():
            spec_b = dataclasses.replace(spec, N=batch)
            inp = synth.make_inputs(spec_b)
            pat = parity.oracle_pattern(inp)
            wb = synth.bf16_bits(inp.w)
            m = masks.mask_from_pattern(pat, wb.shape)
            xb = synth.bf16_bits(inp.x)
            t0 = time.perf_counter()
            conv2d_f64(parity.oracle_shape(spec_b), xb, wb, mask=m, bias=inp.bias.numpy())
            secs += time.perf_counter() - t0
            flops += spec_b.dense_equiv_flops
        return flops, secs

    f1, s1 = run(1)
    batch = 1
    for b in (32, 16, 8, 4, 2):
        if s1 * b <= target_seconds * 1.5:
            batch = b
            break
    flops, secs = (f1, s1) if batch == 1 else run(batch)
    return {"value": flops / secs / 1e12, "unit": "TFLOP/s", "cores": threads(), "kind": "oracle",
            "sample": f"all {len(timed_layers())} layers of the sweep at batch {batch} (of 32), full output tensors, "
                      f"{secs:.1f} s of CPU time", "seconds": secs, "batch": batch}


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import build as oracle_build
    oracle_build.build()
    per_step = max(2.0, min(15.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_leg(per_step)
    vals, secs = [], 0.0
    leg = None
    for _ in range(args.steps):
        leg = oracle_leg(per_step)
        vals.append(leg["value"])
        secs += leg["seconds"]
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU fp64 oracle on host cores, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": leg["cores"], "kind": "oracle",
                         "sample": leg["sample"]},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# DRAM traffic of the sparse forward kernels of one step (7 launches of ssconv_fwd_kernel<sparse> and
# the finishing kernel of the one split layer), dram__bytes_read.sum + dram__bytes_write.sum from an
# ncu capture of this workload (summary and command: profiles/bench_resnet18_sweep_dram_traffic.md).
# It belongs to the kernel sources with the digest below; with other sources the bench reports null.
TRAFFIC_BYTES_PER_STEP = 66.41e6
TRAFFIC_SOURCES = ("forward.cu", "sm100_ptx.cuh", "layout.cuh")
TRAFFIC_SOURCES_SHA256 = "f5473a3b686cfcf438dbd934658b158346017ede67fe2f4402739fec885f9b3f"


def measured_traffic():
    import hashlib
    h = hashlib.sha256()
    root = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2411_00288_b200", "csrc")
    try:
        for name in TRAFFIC_SOURCES:
            with open(os.path.join(root, name), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return TRAFFIC_BYTES_PER_STEP if h.hexdigest() == TRAFFIC_SOURCES_SHA256 else None


# ----------------------------------------------------------------------------- conv stack, end to end
def stack_arm(args):
    """ResNet-50-shaped convolution stack (dense stem, max-pool, 52 masked convolutions) at batch 256
    per GPU: images per second of the whole stack, recorded into one CUDA graph and replayed, with
    the same stack on the dense kernel for comparison.  One JSON line on rank 0."""
    import torch
    import torch.distributed as dist
    from paper_2411_00288_b200 import api, synth, stack, ranks, build as libbuild

    rank, local_rank, world = ranks.env_ranks()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        libbuild.build()
    if world > 1:
        dist.barrier()
    api.lib()
    batch = args.batch or 256
    steps_def = synth.resnet50_stack(batch, residual=args.residual)
    net = stack.ConvStack(steps_def, dev, with_dense=True)
    g = torch.Generator().manual_seed(synth.SEED_BASE + 577 + rank)
    x = torch.zeros((batch, 224, 224, 8), dtype=torch.bfloat16)
    x[..., :3] = torch.randn((batch, 224, 224, 3), generator=g, dtype=torch.float32).to(torch.bfloat16)
    xd = x.to(dev)
    warmup, steps = max(3, args.warmup), min(args.steps, 200)

    def timed(sparse):
        for _ in range(2):
            net.forward(xd, sparse=sparse)
        torch.cuda.synchronize()
        c0 = api.ssconv_launch_count()
        net.forward(xd, sparse=sparse)
        launches = api.ssconv_launch_count() - c0
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            net.forward(xd, sparse=sparse)
        for _ in range(warmup):
            graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return ranks.max_over_ranks(e0.elapsed_time(e1) / steps, dev), launches

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_sparse, launches = timed(True)
    ms_dense, _ = timed(False)
    clocks = sampler.stop() if rank == 0 else None
    status = int(net.status.item())
    if rank == 0:
        flops = net.conv_flops()
        print(json.dumps({
            "metric": "end-to-end images/s of the ResNet-50-shaped convolution stack, 2:4 masked (bf16)",
            "value": ranks.job_throughput(batch, world, ms_sparse), "unit": "images/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_sparse, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD + ("_with_skip_connections" if args.residual else ""),
                       "batch_per_gpu": batch,
                       "stack": "stem 7x7 s2 (dense, input padded 3 -> 8 channels), 3x3 s2 max-pool, 16 "
                                "bottlenecks as reduce -> 3x3 -> expand with bias + ReLU, 4 downsample convolutions on "
                                "their block's input; " + ("skip connections fused into the expand convolutions"
                                                            if args.residual else "no residual additions"),
                       "l2": "activations of a step total several GB (> L2)",
                       "launch": "the stack's calls recorded into one CUDA graph and replayed"},
            "dense_equiv_tflops": ranks.job_throughput(flops, world, ms_sparse) / 1e12,
            "x_dense": ms_dense / ms_sparse, "ms_per_step_dense": ms_dense,
            "images_per_s_dense": ranks.job_throughput(batch, world, ms_dense),
            "gpu_launches": steps * launches, "clocks": clocks, "dev_status": status}))
    if world > 1:
        dist.destroy_process_group()


def train_arm(args):
    """One mask-learning step per layer of the chosen layer set (Sec. 3.1): soft mask -> dense forward
    with the effective weights -> weight gradient -> gradient of the choice weights -> AdamW on them,
    with a seeded stand-in for the loss gradient.  Dense-equivalent TFLOP/s over the two convolutions' FLOPs, and a
    per-layer table of the four kernels' device times.  One JSON line on rank 0."""
    import torch
    import torch.distributed as dist
    from paper_2411_00288_b200 import api, synth, ranks, build as libbuild

    rank, local_rank, world = ranks.env_ranks()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        libbuild.build()
    if world > 1:
        dist.barrier()
    api.lib()
    peaks = load_peaks()
    tau = 0.5
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    prep = []
    for spec in timed_layers():
        inp = synth.make_inputs(spec)
        tr = synth.make_train_inputs(spec)
        desc = api.desc_from_spec(spec)
        need = api.ssconv_wgrad_ws_bytes(desc)
        prep.append(dict(
            spec=spec, desc=desc, x=inp.x.to(dev), w=inp.w.to(dev), bias=inp.bias.to(dev),
            logits=tr.logits.to(dev), noise=tr.noise.to(dev), dy=tr.dy.to(dev),
            z=torch.empty((spec.G, 6), dtype=torch.float32, device=dev), w_eff=torch.empty_like(inp.w, device=dev),
            y=torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=dev),
            dw=torch.empty((spec.C_out, spec.KH, spec.KW, spec.C_in), dtype=torch.float32, device=dev),
            ws=torch.empty((max(need, 16),), dtype=torch.uint8, device=dev),
            gl=torch.empty((spec.G, 6), dtype=torch.float32, device=dev),
            m=torch.zeros((spec.G, 6), dtype=torch.float32, device=dev),
            v=torch.zeros((spec.G, 6), dtype=torch.float32, device=dev)))

    kernels = {
        "soft_mask": lambda L: api.ssconv_soft_mask(L["logits"], L["noise"], tau, L["w"], z=L["z"], w_eff=L["w_eff"]),
        "forward": lambda L: api.ssconv_forward_dense(L["desc"], L["x"], L["w_eff"], L["bias"], y=L["y"],
                                                      dev_status=status),
        "wgrad": lambda L: api.ssconv_wgrad(L["desc"], L["x"], L["dy"], dw=L["dw"], ws=L["ws"], dev_status=status),
        "mask_grad": lambda L: api.ssconv_mask_grad(L["z"], tau, L["w"], L["dw"], g_logits=L["gl"]),
        # (a small learning rate: the timed replays repeat the update hundreds of times on the same gradient)
        "adamw": lambda L: api.ssconv_adamw(L["logits"], L["gl"], L["m"], L["v"], 1, lr=1e-3),
    }

    if args.only_layer is not None:  # profiling aid: the weight gradient of one layer, launched repeatedly
        L = prep[args.only_layer]
        for _ in range(args.layer_iters):
            kernels["wgrad"](L)
        torch.cuda.synchronize()
        print(json.dumps({"only_layer": L["spec"].name, "kernel": "wgrad", "launches": args.layer_iters,
                          "dev_status": int(status.item())}))
        return

    def step():
        for L in prep:
            for k in kernels.values():
                k(L)

    warmup, steps = max(3, args.warmup), min(args.steps, 2000)
    c0 = api.ssconv_launch_count()
    step()
    launches = api.ssconv_launch_count() - c0
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()

    def replay_ms(fn, reps):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return ranks.max_over_ranks(e0.elapsed_time(e1) / reps, dev)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_step = replay_ms(step, steps)
    clocks = sampler.stop() if rank == 0 else None
    per_layer = []
    iters = 50
    for L in prep:
        spec = L["spec"]
        row = {"layer": spec.name}
        for name, k in kernels.items():
            row["us_" + name] = round(replay_ms(lambda: [k(L) for _ in range(iters)], 5) / iters * 1e3, 2)
        row["wgrad_tflops"] = round(spec.dense_equiv_flops / row["us_wgrad"] / 1e6, 1)
        row["wgrad_frac_of_dense_peak"] = round(row["wgrad_tflops"] / peaks["bf16_tflops"], 4)
        # soft_mask moves 88 bytes per group (logits, noise, weights in; z, effective weights out),
        # mask_grad 72 (z, weights, weight gradient in; logit gradient out)
        row["soft_mask_gbs"] = round(88 * spec.G / row["us_soft_mask"] / 1e3, 1)
        row["mask_grad_gbs"] = round(72 * spec.G / row["us_mask_grad"] / 1e3, 1)
        row["adamw_gbs"] = round(28 * 6 * spec.G / row["us_adamw"] / 1e3, 1)
        per_layer.append(row)
    # the two elementwise kernels on as many groups as a whole ResNet-50 has (5.9 M: 0.5 GB of
    # traffic, beyond L2), where their HBM roofline applies
    Gb = 5_900_000
    gen = torch.Generator().manual_seed(synth.SEED_BASE + 4711)
    big = dict(logits=torch.randn((Gb, 6), generator=gen).to(dev), noise=torch.randn((Gb, 6), generator=gen).to(dev),
               w=torch.randn((Gb, 4), generator=gen).to(torch.bfloat16).to(dev),
               dw=torch.randn((Gb, 4), generator=gen).to(dev),
               z=torch.empty((Gb, 6), dtype=torch.float32, device=dev),
               w_eff=torch.empty((Gb, 4), dtype=torch.bfloat16, device=dev),
               gl=torch.randn((Gb, 6), generator=gen).to(dev),
               m=torch.zeros((Gb, 6), dtype=torch.float32, device=dev),
               v=torch.zeros((Gb, 6), dtype=torch.float32, device=dev))
    us_sm = replay_ms(lambda: [api.ssconv_soft_mask(big["logits"], big["noise"], tau, big["w"], z=big["z"],
                                                    w_eff=big["w_eff"]) for _ in range(10)], 5) / 10 * 1e3
    us_mg = replay_ms(lambda: [api.ssconv_mask_grad(big["z"], tau, big["w"], big["dw"], g_logits=big["gl"])
                               for _ in range(10)], 5) / 10 * 1e3
    us_ad = replay_ms(lambda: [api.ssconv_adamw(big["logits"], big["gl"], big["m"], big["v"], 1, lr=1e-3)
                               for _ in range(10)], 5) / 10 * 1e3
    # the norms of Sec. 3.2 over the same number of groups, as one matrix of 2048 rows (9 bytes per group)
    rows_n = 2048
    Gn = Gb // rows_n * rows_n
    pat_n = torch.randint(0, 6, (Gn,), generator=gen, dtype=torch.int64).to(torch.uint8).to(dev)
    w_n = big["w"][:Gn].reshape(rows_n, -1).contiguous()
    out_n = torch.empty((3,), dtype=torch.float32, device=dev)
    us_nm = replay_ms(lambda: [api.ssconv_mask_norms(w_n, pat_n, out=out_n) for _ in range(10)], 5) / 10 * 1e3
    elementwise = {"groups": Gb, "us_soft_mask": round(us_sm, 1), "us_mask_grad": round(us_mg, 1),
                   "us_mask_norms": round(us_nm, 1), "mask_norms_gbs": round(9 * Gn / us_nm / 1e3, 1),
                   "us_adamw": round(us_ad, 1), "adamw_gbs": round(28 * 6 * Gb / us_ad / 1e3, 1),
                   "adamw_frac_of_hbm_peak": round(28 * 6 * Gb / us_ad / 1e3 / peaks["hbm_gbs"], 4),
                   "soft_mask_gbs": round(88 * Gb / us_sm / 1e3, 1), "mask_grad_gbs": round(72 * Gb / us_mg / 1e3, 1),
                   "soft_mask_frac_of_hbm_peak": round(88 * Gb / us_sm / 1e3 / peaks["hbm_gbs"], 4),
                   "mask_grad_frac_of_hbm_peak": round(72 * Gb / us_mg / 1e3 / peaks["hbm_gbs"], 4),
                   "bytes_per_group": {"soft_mask": 88, "mask_grad": 72, "adamw": 168}}
    flops = 2 * sum(L["spec"].dense_equiv_flops for L in prep)
    if rank == 0:
        wg_ms = sum(r["us_wgrad"] for r in per_layer) * 1e-3
        wg_tflops = sum(L["spec"].dense_equiv_flops for L in prep) / (wg_ms * 1e-3) / 1e12
        print(json.dumps({
            "metric": "TFLOP/s of one mask-learning step per layer (dense forward with soft-masked weights + weight "
                      "gradient; bf16, fp32 accumulate)",
            "value": ranks.job_throughput(flops, world, ms_step) / 1e12, "unit": "TFLOP/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD + "_mask_learning_step", "layers": len(prep), "tau": tau,
                       "batch_per_gpu": prep[0]["spec"].N,
                       "launch": "the step's C-ABI calls recorded into one CUDA graph and replayed",
                       "l2": "one buffer set (the step's tensors total more than L2 only for the larger layer sets)"},
            "roofline": {"bound": "tensor", "kernel": "ssconv_wgrad_kernel", "achieved": wg_tflops,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": wg_tflops / peaks["bf16_tflops"],
                         "peak_source": f"dense bf16 burst of {peaks['source']} peaks", "traffic": None},
            "per_layer": per_layer, "elementwise_at_resnet50_size": elementwise,
            "gpu_launches": steps * launches, "clocks": clocks, "dev_status": int(status.item())}))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- GPU arm
def main():
    global CONFIG_ID, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layer-iters", type=int, default=200)
    ap.add_argument("--only-layer", type=int, default=None,
                    help="profiling aid: launch just this layer of the sweep --layer-iters times and exit")
    ap.add_argument("--dense", action="store_true", help="with --only-layer: use the dense kernel")
    ap.add_argument("--residual", action="store_true",
                    help="with --workload-config 5: fuse the network's skip connections into the expand convolutions")
    ap.add_argument("--train", action="store_true",
                    help="time one mask-learning step per layer (soft mask, dense forward, weight gradient, "
                         "choice-weight gradient) instead of the inference sweep")
    ap.add_argument("--batch", type=int, default=None, help="with --workload-config 5: images per GPU (default 256)")
    ap.add_argument("--workload-config", type=int, default=CONFIG_ID, choices=sorted(WORKLOADS),
                    help="layer set to run (default: the benchmarked ResNet-18 sweep)")
    args = ap.parse_args()
    CONFIG_ID = args.workload_config
    WORKLOAD = WORKLOADS[CONFIG_ID]
    if args.impl == "reference":
        reference_arm(args)
        return
    if CONFIG_ID == 5:
        stack_arm(args)
        return
    if args.train:
        train_arm(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2411_00288_b200 import api, synth, ranks, build as libbuild

    rank, local_rank, world = ranks.env_ranks()
    distributed = world > 1
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if distributed:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        libbuild.build()
    if distributed:
        dist.barrier()
    api.lib()
    peaks = load_peaks()
    warmup = max(3, args.warmup)

    layers = timed_layers()
    if args.only_layer is not None:
        layers = [layers[args.only_layer]]
    # ---- one-off preparation with the library's own kernels: select -> compress (S1, S2)
    prep = []
    set_bytes = sum(2 * (s.N * s.H * s.W * s.C_in + s.P * s.C_out) for s in layers)
    n_sets = max(2, -(-int(1.5 * L2_BYTES) // set_bytes) + 1)
    t_prep0 = time.perf_counter()
    for spec in layers:
        inp = synth.make_inputs(spec)
        desc = api.desc_from_spec(spec)
        w = inp.w.to(dev)
        bias = inp.bias.to(dev)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        xs = [inp.x.to(dev)]
        for r in range(1, n_sets):
            xs.append(synth.make_inputs(spec, seed=spec.seed + 7919 * r, x_only=True).x.to(dev))
        ys = [torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=dev)
              for _ in range(n_sets)]
        prep.append(dict(spec=spec, desc=desc, w=w, bias=bias, w_comp=w_comp, meta=meta, xs=xs, ys=ys,
                         x_host=inp.x.pin_memory(),
                         y_host=torch.empty(ys[0].shape, dtype=torch.bfloat16).pin_memory()))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    prep_seconds = time.perf_counter() - t_prep0

    if args.only_layer is not None:
        L = prep[0]
        for i in range(args.layer_iters):
            r = i % n_sets
            if args.dense:
                api.ssconv_forward_dense(L["desc"], L["xs"][r], L["w"], L["bias"], y=L["ys"][r], dev_status=status)
            else:
                api.ssconv_forward(L["desc"], L["xs"][r], L["w_comp"], L["meta"], L["bias"], y=L["ys"][r],
                                   dev_status=status)
        torch.cuda.synchronize()
        print(json.dumps({"only_layer": L["spec"].name, "launches": args.layer_iters, "dense": args.dense,
                          "dev_status": int(status.item())}))
        return

    def step(r, sparse=True):
        for L in prep:
            if sparse:
                api.ssconv_forward(L["desc"], L["xs"][r], L["w_comp"], L["meta"], L["bias"], y=L["ys"][r],
                                   dev_status=status)
            else:
                api.ssconv_forward_dense(L["desc"], L["xs"][r], L["w"], L["bias"], y=L["ys"][r], dev_status=status)

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return ranks.max_over_ranks(ms, dev)

    def capture(fn):
        """Record fn()'s launches into a CUDA graph (the launches are the same C-ABI calls; the
        graph only removes the host-side launch cost from the timed region)."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    def time_replays(graphs, replays):
        """Replay graphs[i % len] for i < replays between two events; max over ranks, in ms."""
        if not isinstance(graphs, (list, tuple)):
            graphs = [graphs]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for i in range(replays):
            graphs[i % len(graphs)].replay()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1))

    # eager warm-up (also performs every one-time host set-up before any capture)
    launches_per_step = 0
    for i in range(warmup):
        c0 = api.ssconv_launch_count()
        step(i % n_sets, True)
        launches_per_step = api.ssconv_launch_count() - c0
        step(i % n_sets, False)
    torch.cuda.synchronize()

    # one graph per buffer set = one step; step i replays graph i % n_sets
    g_sparse = [capture(lambda r=r: step(r, True)) for r in range(n_sets)]
    g_dense = [capture(lambda r=r: step(r, False)) for r in range(n_sets)]
    total_flops = sum(s.dense_equiv_flops for s in layers)
    steps = args.steps
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    time_replays(g_sparse, warmup)
    ms_total = time_replays(g_sparse, steps)
    ms_per_step = ms_total / steps
    value = ranks.job_throughput(total_flops, world, ms_per_step) / 1e12

    # ---- dense counterpart (S4) on the same buffers, same rotation
    time_replays(g_dense, warmup)
    ms_dense = time_replays(g_dense, steps) / steps
    clocks = sampler.stop() if rank == 0 else None

    # ---- per-layer device times: a graph of `layer_iters` back-to-back launches of one layer,
    # rotating buffer sets, timed with events on the launching stream
    per_layer = []
    sum_kernel_ms = 0.0
    sum_roof_ms = 0.0
    sparse_peak = 2.0 * peaks["bf16_tflops"]
    for L in prep:
        spec = L["spec"]
        res = {}
        for sparse in (True, False):
            def many(L=L, sparse=sparse):
                for i in range(args.layer_iters):
                    r = i % n_sets
                    if sparse:
                        api.ssconv_forward(L["desc"], L["xs"][r], L["w_comp"], L["meta"], L["bias"], y=L["ys"][r],
                                           dev_status=status)
                    else:
                        api.ssconv_forward_dense(L["desc"], L["xs"][r], L["w"], L["bias"], y=L["ys"][r],
                                                 dev_status=status)
            g = capture(many)
            time_replays(g, 1)
            res[sparse] = time_replays(g, 5) / (5 * args.layer_iters)
            del g
        t_s, t_d = res[True], res[False]
        flops = spec.dense_equiv_flops
        bytes_alg = spec.algorithmic_bytes(sparse=True)
        t_c = flops / (sparse_peak * 1e12) * 1e3
        t_m = bytes_alg / (peaks["hbm_gbs"] * 1e9) * 1e3
        roof = max(t_c, t_m)
        sum_kernel_ms += t_s
        sum_roof_ms += roof
        per_layer.append({"layer": spec.name, "us_sparse": round(t_s * 1e3, 2), "us_dense": round(t_d * 1e3, 2),
                          "tflops": round(flops / t_s / 1e9, 1), "gbs": round(bytes_alg / t_s / 1e6, 1),
                          "bound": "tensor" if t_c >= t_m else "hbm", "us_roofline": round(roof * 1e3, 2),
                          "roofline_frac": round(roof / t_s, 4), "x_dense": round(t_d / t_s, 3),
                          "plan": api.ssconv_plan(L["desc"], True)})

    # ---- end to end through the public API with host buffers: every step copies each layer's input
    # from pinned host memory, runs the layer, and copies its output back.  Three streams (copy in,
    # compute, copy out) chained by events, so that the copies of one layer overlap the kernels
    # and the opposite-direction copies of its neighbours, as a serving loop would do it.
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in prep]
    ev_run = [torch.cuda.Event() for _ in prep]
    ev_out = [torch.cuda.Event() for _ in prep]

    def e2e_step(first):
        for i, L in enumerate(prep):
            with torch.cuda.stream(s_in):
                if not first:
                    s_in.wait_event(ev_run[i])   # the previous step's kernel has read this input buffer
                L["xs"][0].copy_(L["x_host"], non_blocking=True)
                ev_in[i].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[i])
                if not first:
                    s_run.wait_event(ev_out[i])  # the previous step's copy-out has read this output buffer
                api.ssconv_forward(L["desc"], L["xs"][0], L["w_comp"], L["meta"], L["bias"], y=L["ys"][0],
                                   dev_status=status)
                ev_run[i].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[i])
                L["y_host"].copy_(L["ys"][0], non_blocking=True)
                ev_out[i].record(s_out)

    torch.cuda.synchronize()
    for it in range(3):
        e2e_step(it == 0)
    torch.cuda.synchronize()
    k_e2e = 20
    e2e_t0, e2e_t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e2e_t0.record(s_in)
    for _ in range(k_e2e):
        e2e_step(False)
    s_out.wait_stream(s_run)
    s_out.wait_stream(s_in)
    e2e_t1.record(s_out)
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(e2e_t0.elapsed_time(e2e_t1) / k_e2e)
    h2d = sum(L["x_host"].numel() * 2 for L in prep)
    d2h = sum(L["y_host"].numel() * 2 for L in prep)
    dev_status = int(status.item())

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import build as oracle_build
        oracle_build.build()
        leg = oracle_leg(15.0)
        cpu = {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        achieved = total_flops / (sum_kernel_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "layers": len(layers), "batch_per_gpu": layers[0].N,
                       "l2": f"rotating {n_sets} buffer sets of {set_bytes / 2**20:.0f} MiB (> L2) per rank",
                       "masks": "magnitude top-2 of 4, selected and compressed once before timing",
                       "launch": "the C-ABI calls of one step recorded into a CUDA graph per buffer set and replayed",
                       "one_off_prepare_s": round(prep_seconds, 3)},
            "x_dense": ms_dense / ms_per_step, "ms_per_step_dense": ms_dense,
            "roofline": {"bound": "tensor", "kernel": "ssconv_fwd_kernel<sparse>", "achieved": achieved,
                         "peak": sparse_peak, "unit": "TFLOP/s", "frac": achieved / sparse_peak,
                         "peak_source": f"2 x dense bf16 burst of {peaks['source']} peaks (nominal sparse:dense ratio)",
                         "layer_mix_ceiling": total_flops / (sum_roof_ms * 1e-3) / 1e12,
                         "frac_of_layer_mix_ceiling": sum_roof_ms / sum_kernel_ms,
                         "hbm_peak_gbs": peaks["hbm_gbs"],
                         "traffic": measured_traffic() if CONFIG_ID == 2 else None,
                         "traffic_unit": "bytes per step (DRAM read + write of the sparse forward and finishing "
                                         "kernels, ncu)",
                         "algorithmic_bytes_per_step": sum(L["spec"].algorithmic_bytes(sparse=True) for L in prep)},
            "per_layer": per_layer,
            "e2e": {"value": world * total_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": steps * launches_per_step,
            "clocks": clocks, "dev_status": dev_status,
        }
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
