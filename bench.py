#!/usr/bin/env python
"""Benchmark of the 2:4 sparse convolution forward on B200.

Default workload: the convolution stack of a Torchvision-shaped ResNet-50 at batch 256 per GPU
(the largest configuration: a dense 7x7 stem on 3-channel images, a 3x3 max-pool and 52 masked
convolutions; seeded synthetic images and weights, masks by magnitude, selected and compressed
once beforehand with the library's own kernels).  A step is one forward pass of the whole stack.
The reported value is dense-equivalent TFLOP/s (2*P*C_out*K per convolution, the stem counted with
its 3 real input channels) over all ranks; images per second, the dense counterpart, a per-layer
table with each layer's roofline, the end-to-end figure with host buffers, the CPU oracle and
short summaries of the three per-layer sweeps (ResNet-18 3x3 sweep, ResNet-50 bottleneck layers,
ConvNeXt-T point-wise layers) ride in the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload-config 2|3|4|5] [--train]

Prints exactly one JSON line on rank 0.  With --gpus N > 1 and no torchrun environment it starts N
ranks itself (one per GPU; the ranks share nothing but the timing barrier).
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
CONFIG_ID = 5          # the benchmarked workload; --workload-config picks one of the per-layer sweeps instead
WORKLOAD = WORKLOADS[CONFIG_ID]
MIN_REGIONS = 30       # timed regions of --steps steps each; the median is reported


# DRAM bytes of one step of the stack at batch 256, from the ncu counters summarised in
# profiles/bench_resnet50_stack_dram_traffic.md; valid for the kernels whose sources hash to `sources`
# (anything else reports null: the counters would have to be taken again).
STACK_TRAFFIC = {"batch": 256, "read": 4516161792, "write": 5831267328, "sources": "97ecc4868de1270a"}
TRAFFIC_SOURCES = ("paper_2411_00288_b200/csrc/forward.cu", "paper_2411_00288_b200/csrc/pool.cu",
                   "paper_2411_00288_b200/csrc/sm100_ptx.cuh", "paper_2411_00288_b200/csrc/layout.cuh",
                   "paper_2411_00288_b200/stack.py")


def stack_traffic(batch, residual):
    """Measured DRAM bytes per step, or None when the measured kernels are not the ones in the tree."""
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, f), "rb") as fh:
            h.update(fh.read())
    if batch != STACK_TRAFFIC["batch"] or residual or h.hexdigest()[:16] != STACK_TRAFFIC["sources"]:
        return None
    return STACK_TRAFFIC["read"] + STACK_TRAFFIC["write"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return {"hbm_gbs": float(pk["hbm_gbs"]), "bf16_tflops": float(pk["bf16_tflops"]),
                "bf16_tflops_sustained": float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def timed_layers(config_id=None):
    from paper_2411_00288_b200 import synth
    return [s for s in synth.config_layers(CONFIG_ID if config_id is None else config_id) if not s.extra]


def spread(values):
    """Median, extremes and the 10th / 90th percentiles of a list of region times."""
    v = sorted(values)
    n = len(v)
    return {"median": statistics.median(v), "min": v[0], "max": v[-1], "p10": v[int(0.1 * (n - 1))],
            "p90": v[int(round(0.9 * (n - 1)))], "regions": n}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the benchmark runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None
        self.marks = {}

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

    def mark(self, name):
        """Remember how many samples had arrived when leg `name` started."""
        self.marks[name] = len(self.lines)

    def _summary(self, lines):
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # samples taken while the GPU was working (an idle GPU drops its clock between legs)
        busy = [c for c, w in zip(sm, power) if w >= 0.5 * max(power)] if power else []
        return {"sm_mhz": statistics.median(busy) if busy else (statistics.median(sm) if sm else None),
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "samples_under_load": len(busy),
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons)}

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)   # one more sampling period
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        out = self._summary(self.lines)
        bounds = sorted(self.marks.items(), key=lambda kv: kv[1]) + [("end", len(self.lines))]
        out["legs"] = {}
        for (name, lo), (_, hi) in zip(bounds, bounds[1:]):
            leg = self._summary(self.lines[lo:hi])
            out["legs"][name] = {k: leg[k] for k in ("sm_mhz", "samples", "reasons")}
        return out


# ----------------------------------------------------------------------------- CPU oracle leg
_ORACLE_WEIGHTS = {}


def stack_conv_specs(batch):
    """The 53 convolutions of the benchmarked stack at the given batch: (spec, masked?)."""
    from paper_2411_00288_b200 import synth
    return [(st.spec, st.kind == "conv") for st in synth.resnet50_stack(batch) if st.kind != "maxpool"]


def stack_flops(batch):
    """Dense-equivalent FLOPs of one pass: 2*P*C_out*K per convolution; the stem with its 3 real channels."""
    total = 0
    for spec, masked in stack_conv_specs(batch):
        total += spec.dense_equiv_flops if masked else spec.dense_equiv_flops * 3 // spec.C_in
    return total


def oracle_leg(target_seconds: float = 15.0, config_id=None):
    """Time the fp64 CPU oracle, as it stands, on a bounded sample of the same workload: every
    convolution of the workload on seeded inputs of its own shape, full output tensors, at the largest
    batch that keeps the leg near `target_seconds`."""
    import dataclasses
    from oracle import masks
    from oracle.conv import conv2d_f64, threads
    from paper_2411_00288_b200 import synth
    from tests import parity

    cfg = CONFIG_ID if config_id is None else config_id
    full_batch = {2: 32, 3: 64, 4: 128, 5: 256}[cfg]

    def layer_list(batch):
        if cfg == 5:
            return stack_conv_specs(batch)
        return [(dataclasses.replace(s, N=batch), True) for s in timed_layers(cfg)]

    def run(batch):
        flops, secs = 0, 0.0
        for idx, (spec, masked) in enumerate(layer_list(batch)):
            key = (cfg, idx)
            if key not in _ORACLE_WEIGHTS:   # weights, mask and bias do not depend on the batch: drawn once
                inp = synth.make_inputs(dataclasses.replace(spec, N=1))
                wb = synth.bf16_bits(inp.w)
                m = masks.mask_from_pattern(parity.oracle_pattern(inp), wb.shape) if masked else None
                _ORACLE_WEIGHTS[key] = (wb, m, inp.bias.numpy())
            wb, m, bias = _ORACLE_WEIGHTS[key]
            xb = synth.bf16_bits(synth.make_inputs(spec, x_only=True).x)
            t0 = time.perf_counter()
            conv2d_f64(parity.oracle_shape(spec), xb, wb, mask=m, bias=bias)
            secs += time.perf_counter() - t0
            flops += spec.dense_equiv_flops if masked else spec.dense_equiv_flops * 3 // spec.C_in
        return flops, secs

    f1, s1 = run(1)
    batch = 1
    for b in (32, 16, 8, 4, 2):
        if b <= full_batch and s1 * b <= target_seconds * 1.5:
            batch = b
            break
    flops, secs = (f1, s1) if batch == 1 else run(batch)
    what = ("the 53 convolutions of the stack" if cfg == 5 else f"all {len(layer_list(1))} layers of the sweep")
    return {"value": flops / secs / 1e12, "unit": "TFLOP/s", "cores": threads(), "kind": "oracle",
            "sample": f"{what} at batch {batch} (of {full_batch}), each on seeded inputs of its own shape, full "
                      f"output tensors, {secs:.1f} s of CPU time",
            "seconds": secs, "batch": batch, "images_per_s": batch / secs if cfg == 5 else None}


def reference_arm(args):
    """The reference arm: the fp64 CPU oracle as it stands (the paper publishes no code to install), on
    the same workload, metric and unit; each step is a bounded sample of it."""
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


# ----------------------------------------------------------------------------- timing helpers
class Timer:
    """CUDA-event timing of graph replays on the current stream, with the barrier / synchronise
    bracket and the maximum over ranks."""

    def __init__(self, torch, dist, ranks, dev, distributed):
        self.torch, self.dist, self.ranks, self.dev, self.distributed = torch, dist, ranks, dev, distributed

    def barrier(self):
        if self.distributed:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def capture(self, fn):
        """Record fn()'s launches into a CUDA graph (the launches are the same C-ABI calls; the graph
        only removes the host-side launch cost from the timed region)."""
        g = self.torch.cuda.CUDAGraph()
        with self.torch.cuda.graph(g):
            fn()
        return g

    def region(self, graphs, replays):
        """Replay graphs[i % len] for i < replays between two events; max over ranks, in ms."""
        if not isinstance(graphs, (list, tuple)):
            graphs = [graphs]
        e0 = self.torch.cuda.Event(enable_timing=True)
        e1 = self.torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for i in range(replays):
            graphs[i % len(graphs)].replay()
        e1.record()
        self.barrier()
        return self.ranks.max_over_ranks(e0.elapsed_time(e1), self.dev)

    def regions(self, graphs, replays, count, budget_s=20.0):
        """`count` regions of `replays` replays each (fewer if they would outlast the budget, never
        fewer than 5); per-replay times in ms."""
        out = []
        t0 = time.perf_counter()
        for i in range(count):
            out.append(self.region(graphs, replays) / replays)
            if i >= 4 and time.perf_counter() - t0 > budget_s:
                break
        return out


def layer_roofline(spec, peaks, sparse=True, real_c_in=None):
    """(flops, algorithmic bytes, compute roofline ms, memory roofline ms) of one convolution.  The
    compute peak is 2 x the measured dense bf16 burst for a 2:4 layer (nominal sparse : dense ratio),
    the measured dense burst for a dense one; the memory peak is the measured HBM copy bandwidth."""
    flops = spec.dense_equiv_flops
    bytes_alg = spec.algorithmic_bytes(sparse=sparse)
    if real_c_in is not None:   # channel-padded input: count the real channels
        flops = flops * real_c_in // spec.C_in
        bytes_alg -= 2 * spec.N * spec.H * spec.W * (spec.C_in - real_c_in)
        bytes_alg -= 2 * spec.C_out * spec.KH * spec.KW * (spec.C_in - real_c_in)
    peak = (2.0 if sparse else 1.0) * peaks["bf16_tflops"]
    return flops, bytes_alg, flops / (peak * 1e12) * 1e3, bytes_alg / (peaks["hbm_gbs"] * 1e9) * 1e3


# ----------------------------------------------------------------------------- per-layer sweeps (configs 2-4)
def sweep_measure(cfg, api, synth, torch, tm, dev, peaks, l2_bytes, steps, regions, layer_iters, status,
                  only_layer=None, want_e2e=False):
    """One of the per-layer workloads: every layer on its own seeded input (rotating over buffer sets
    larger than L2), a step = all layers once; the dense counterpart; per-layer device times and
    rooflines.  Returns a dict; the caller formats it."""
    layers = timed_layers(cfg)
    if only_layer is not None:
        layers = [layers[only_layer]]
    set_bytes = sum(2 * (s.N * s.H * s.W * s.C_in + s.P * s.C_out) for s in layers)
    n_sets = max(2, -(-int(1.5 * l2_bytes) // set_bytes) + 1)
    prep = []
    t_prep0 = time.perf_counter()
    gen = torch.Generator(device=dev).manual_seed(synth.SEED_BASE + 31 * cfg)
    for spec in layers:
        inp = synth.make_inputs(spec)
        desc = api.desc_from_spec(spec)
        w = inp.w.to(dev)
        bias = inp.bias.to(dev)
        if spec.mask_source == "gumbel_logits":
            pat = api.ssconv_select_mask(api.MASK_LOGITS_F32, inp.scores.to(dev), spec.G)
        else:
            pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        fold = api.ssconv_fold_factor(desc)
        if fold > 1:   # few output channels: neighbouring output pixels as extra output channels, same bytes out
            w, bias_f = api.ssconv_fold_weights(desc, fold, w, bias)
            pat, _ = api.ssconv_fold_weights(desc, fold, pat)
            desc, bias = api.ssconv_fold_desc(desc, fold), bias_f
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        xs = [inp.x.to(dev)]
        for _ in range(1, n_sets):   # further buffer sets only rotate the traffic: drawn on the device
            xs.append(torch.randn(inp.x.shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16))
        ys = [torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=dev)
              for _ in range(n_sets)]
        entry = dict(spec=spec, desc=desc, w=w, bias=bias, w_comp=w_comp, meta=meta, xs=xs, ys=ys, fold=fold)
        if want_e2e:
            entry["x_host"] = inp.x.pin_memory()
            entry["y_host"] = torch.empty(ys[0].shape, dtype=torch.bfloat16).pin_memory()
        prep.append(entry)
    torch.cuda.synchronize()
    prep_seconds = time.perf_counter() - t_prep0

    def call(L, r, sparse):
        if sparse:
            api.ssconv_forward(L["desc"], L["xs"][r], L["w_comp"], L["meta"], L["bias"], y=L["ys"][r], dev_status=status)
        else:
            api.ssconv_forward_dense(L["desc"], L["xs"][r], L["w"], L["bias"], y=L["ys"][r], dev_status=status)

    def step(r, sparse=True):
        for L in prep:
            call(L, r, sparse)

    launches_per_step = 0
    for i in range(3):   # eager warm-up (also performs every one-time host set-up before any capture)
        c0 = api.ssconv_launch_count()
        step(i % n_sets, True)
        launches_per_step = api.ssconv_launch_count() - c0
        step(i % n_sets, False)
    torch.cuda.synchronize()
    g_sparse = [tm.capture(lambda r=r: step(r, True)) for r in range(n_sets)]
    g_dense = [tm.capture(lambda r=r: step(r, False)) for r in range(n_sets)]
    tm.region(g_sparse, 2 * n_sets)
    ms_sparse = tm.regions(g_sparse, steps, regions, budget_s=8.0)
    tm.region(g_dense, 2 * n_sets)
    ms_dense = tm.regions(g_dense, steps, max(5, regions // 3), budget_s=4.0)
    del g_sparse, g_dense

    per_layer, sum_t, sum_roof, sum_t_dense = [], 0.0, 0.0, 0.0
    for L in prep:
        spec = L["spec"]
        res = {}
        for sparse in (True, False):
            g = tm.capture(lambda L=L, sparse=sparse: [call(L, i % n_sets, sparse) for i in range(layer_iters)])
            tm.region(g, 1)
            res[sparse] = min(tm.region(g, 2) / 2 for _ in range(3)) / layer_iters
            del g
        flops, bytes_alg, t_c, t_m = layer_roofline(spec, peaks, sparse=True)
        roof = max(t_c, t_m)
        sum_t += res[True]
        sum_t_dense += res[False]
        sum_roof += roof
        per_layer.append({"layer": spec.name, "us_sparse": round(res[True] * 1e3, 2), "us_dense": round(res[False] * 1e3, 2),
                          "tflops": round(flops / res[True] / 1e9, 1), "gbs": round(bytes_alg / res[True] / 1e6, 1),
                          "bound": "tensor" if t_c >= t_m else "hbm", "us_roofline": round(roof * 1e3, 2),
                          "roofline_frac": round(roof / res[True], 4), "x_dense": round(res[False] / res[True], 3),
                          "plan": dict(api.ssconv_plan(L["desc"], True), fold=L["fold"])})
    total_flops = sum(s.dense_equiv_flops for s in layers)
    out = dict(layers=layers, prep=prep, n_sets=n_sets, set_bytes=set_bytes, prep_seconds=prep_seconds,
               launches_per_step=launches_per_step, ms_sparse=ms_sparse, ms_dense=ms_dense, per_layer=per_layer,
               sum_kernel_ms=sum_t, sum_kernel_ms_dense=sum_t_dense, sum_roof_ms=sum_roof, total_flops=total_flops,
               bytes_alg=sum(s.algorithmic_bytes(sparse=True) for s in layers))
    return out


def sweep_summary(cfg, m, world, ranks):
    """The short form of a sweep for the headline line."""
    ms = statistics.median(m["ms_sparse"])
    return {"workload": WORKLOADS[cfg], "layers": len(m["layers"]), "ms_per_step": round(ms, 5),
            "tflops": round(ranks.job_throughput(m["total_flops"], world, ms) / 1e12, 1),
            "x_dense": round(statistics.median(m["ms_dense"]) / ms, 3),
            "roofline_frac": round(m["sum_roof_ms"] / m["sum_kernel_ms"], 4),
            "min_layer_x_dense": min(r["x_dense"] for r in m["per_layer"]),
            "per_layer": [{k: r[k] for k in ("layer", "us_sparse", "roofline_frac", "x_dense", "bound")}
                          for r in m["per_layer"]]}


def fp8_summary(api, synth, torch, tm, dev, l2_bytes, batch, status):
    """The masked convolutions of the stack on e4m3 operands (ssconv_forward_fp8), layer by layer on seeded
    inputs of each distinct shape, beside the bf16 kernels on the same shapes: device times weighted by how
    often a shape occurs in the stack.  Context for the 8-bit path, not part of the step."""
    shapes = {}
    for spec in synth.config_layers(5, batch):
        if spec.C_in % 16 or spec.extra:
            continue
        key = (spec.H, spec.C_in, spec.C_out, spec.KH, spec.stride)
        shapes.setdefault(key, [spec, 0])[1] += 1
    rows, t_bf16, t_fp8, flops = [], 0.0, 0.0, 0.0
    iters = 10
    for spec, count in shapes.values():
        desc = api.desc_from_spec(spec)
        inp = synth.make_inputs(spec)
        w, bias = inp.w.to(dev), inp.bias.to(dev)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        fold = api.ssconv_fold_factor(desc)
        d16, w16, b16 = desc, w, bias
        if fold > 1:
            w16, b16 = api.ssconv_fold_weights(desc, fold, w, bias)
            pat, _ = api.ssconv_fold_weights(desc, fold, pat)
            d16 = api.ssconv_fold_desc(desc, fold)
        w_comp, meta = api.ssconv_compress(d16, w16, pat)
        wq = api.ssconv_quantize_e4m3(w16, 16.0)
        pq = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, wq, wq.numel() // 4)
        wq_comp, metaq = api.ssconv_compress_fp8(d16, wq, pq)
        set_bytes = spec.N * spec.H * spec.W * spec.C_in * 2 + 2 * spec.P * spec.C_out
        n_sets = min(16, max(2, -(-int(1.5 * l2_bytes) // set_bytes) + 1))
        xs = [inp.x.to(dev)] + [torch.randn(inp.x.shape, device=dev).to(torch.bfloat16) for _ in range(n_sets - 1)]
        xq = [api.ssconv_quantize_e4m3(x, 1.0) for x in xs]
        ys = [torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=dev)
              for _ in range(n_sets)]
        res = {}
        for name, call in (
                ("bf16", lambda r: api.ssconv_forward(d16, xs[r], w_comp, meta, b16, y=ys[r], dev_status=status)),
                ("e4m3", lambda r: api.ssconv_forward_fp8(d16, xq[r], wq_comp, metaq, b16, 1.0 / 16.0, y=ys[r],
                                                          dev_status=status))):
            for r in range(min(3, n_sets)):
                call(r)
            torch.cuda.synchronize()
            g = tm.capture(lambda call=call: [call(i % n_sets) for i in range(iters)])
            tm.region(g, 1)
            res[name] = min(tm.region(g, 2) / 2 for _ in range(3)) / iters
            del g
        t_bf16 += count * res["bf16"]
        t_fp8 += count * res["e4m3"]
        flops += count * spec.dense_equiv_flops
        rows.append({"layer": spec.name, "count": count, "us_bf16": round(res["bf16"] * 1e3, 2),
                     "us_e4m3": round(res["e4m3"] * 1e3, 2),
                     "tflops_e4m3": round(spec.dense_equiv_flops / (res["e4m3"] * 1e-3) / 1e12, 1)})
        del xs, xq, ys
        torch.cuda.empty_cache()
    return {"what": "the stack's masked convolutions on e4m3 activations and weights (fp32 accumulation, bf16 outputs) "
                    "against the bf16 kernels on the same shapes; sums weighted by the shapes' multiplicity",
            "layers": int(sum(c for _, c in shapes.values())), "sum_ms_bf16": round(t_bf16, 4),
            "sum_ms_e4m3": round(t_fp8, 4), "x_bf16": round(t_bf16 / t_fp8, 3),
            "tflops_e4m3": round(flops / (t_fp8 * 1e-3) / 1e12, 1), "per_layer": rows}


def convnext_summary(api, torch, tm, dev, batch=128):
    """A ConvNeXt-T-shaped network chained through the library (convnext.py: patchify stem, 18 blocks of depthwise 7x7
    -> layer norm -> 1x1 2:4 with GELU -> 1x1 2:4 with the skip connection fused, three downsample convolutions), the
    whole forward pass recorded into one CUDA graph.  Context for the other network family of Sec. 4."""
    from paper_2411_00288_b200 import convnext
    net = convnext.ConvNeXtStack(batch, dev)
    x = torch.randn((batch, 224, 224, 3), device=dev).to(torch.bfloat16)
    for sparse in (True, False):
        net.forward(x, sparse)
    torch.cuda.synchronize()
    res = {}
    for sparse in (True, False):
        g = tm.capture(lambda sparse=sparse: net.forward(x, sparse))
        tm.region(g, 2)
        res[sparse] = min(tm.region(g, 5) / 5 for _ in range(3))
        del g
    kinds = {}
    for i, st in enumerate(net.steps):
        g = tm.capture(lambda i=i: [net.run_step(i, x) for _ in range(3)])
        tm.region(g, 1)
        kinds[st.kind] = kinds.get(st.kind, 0.0) + tm.region(g, 2) / 6
        del g
    out = {"what": "ConvNeXt-T-shaped forward pass, 224 x 224 images, all convolutions but the stem and the depthwise ones "
                   "2:4 masked; seeded synthetic weights", "batch": batch, "calls_per_step": len(net.steps),
           "ms_per_step": round(res[True], 4), "images_per_s": round(batch / res[True] * 1e3, 1),
           "x_dense": round(res[False] / res[True], 3),
           "masked_conv_tflops": round(net.masked_conv_flops() / (kinds["conv"] * 1e-3) / 1e12, 1),
           "ms_by_kind": {("masked_conv" if k == "conv" else k): round(v, 4) for k, v in kinds.items()},
           "dev_status": int(net.status.item())}
    del net
    torch.cuda.empty_cache()
    return out


def convnext_arm(args):
    """The ConvNeXt-T-shaped pass on its own (one GPU): prints convnext_summary as one JSON line."""
    import torch
    from paper_2411_00288_b200 import api, ranks, build as libbuild
    libbuild.build()
    api.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    tm = Timer(torch, None, ranks, dev, False)
    print(json.dumps(convnext_summary(api, torch, tm, dev, batch=args.batch or 128)))


# ----------------------------------------------------------------------------- mask-learning step
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
        # the gradient with respect to the layer's input (what chains layers; not part of the step timed above),
        # from the output gradient and the effective weights
        try:
            dws = torch.empty((max(api.ssconv_dgrad_ws_bytes(L["desc"]), 16),), dtype=torch.uint8, device=dev)
            dxb = torch.empty(L["x"].shape, dtype=torch.bfloat16, device=dev)
            row["us_dgrad"] = round(replay_ms(lambda: [api.ssconv_dgrad(L["desc"], L["dy"], L["w_eff"], dx=dxb, ws=dws,
                                                                        dev_status=status) for _ in range(iters)], 5)
                                    / iters * 1e3, 2)
            row["dgrad_tflops"] = round(spec.dense_equiv_flops / row["us_dgrad"] / 1e6, 1)
            del dws, dxb
        except api.SsconvError:
            row["us_dgrad"] = None
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
            "roofline": {"bound": "tensor", "kernel": "ssconv_wgrad_pair_kernel (ssconv_wgrad_kernel on layers of one or two "
                                                        "k-blocks) + the adding kernel", "achieved": wg_tflops,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": wg_tflops / peaks["bf16_tflops"],
                         "peak_source": f"dense bf16 burst of {peaks['source']} peaks", "traffic": None},
            "per_layer": per_layer, "elementwise_at_resnet50_size": elementwise,
            "gpu_launches": steps * launches, "clocks": clocks, "dev_status": int(status.item())}))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- conv stack (the headline)
def stack_arm(args):
    """ResNet-50-shaped convolution stack at batch 256 per GPU, recorded into one CUDA graph and replayed."""
    import torch
    import torch.distributed as dist
    from paper_2411_00288_b200 import api, synth, stack, ranks, build as libbuild

    rank, local_rank, world = ranks.env_ranks()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    distributed = world > 1
    if distributed:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        libbuild.build()
    if distributed:
        dist.barrier()
    api.lib()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()          # before any warm-up: it runs through every leg below
    peaks = load_peaks()
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    tm = Timer(torch, dist, ranks, dev, distributed)
    batch = args.batch or 256
    warmup, steps = max(3, args.warmup), max(1, min(args.steps, 200))

    t_prep0 = time.perf_counter()
    steps_def = synth.resnet50_stack(batch, residual=args.residual)
    net = stack.ConvStack(steps_def, dev, with_dense=True)
    g = torch.Generator().manual_seed(synth.SEED_BASE + 577 + rank)
    x3_host = torch.randn((batch, 224, 224, 3), generator=g, dtype=torch.float32).to(torch.bfloat16).pin_memory()
    x_dev = x3_host.to(dev)   # (the stack takes the 3-channel images as they are: its stem starts with a space-to-depth)
    torch.cuda.synchronize()
    prep_seconds = time.perf_counter() - t_prep0
    act_bytes = sum(o.numel() * 2 for o in net.outputs) + x_dev.numel() * 2

    # ---- the step: whole stack, sparse; then the dense counterpart on the same buffers
    sampler.mark("step")
    for _ in range(2):
        net.forward(x_dev, sparse=True)
        net.forward(x_dev, sparse=False)
    torch.cuda.synchronize()
    c0 = api.ssconv_launch_count()
    net.forward(x_dev, sparse=True)
    launches = api.ssconv_launch_count() - c0
    torch.cuda.synchronize()
    g_sparse = tm.capture(lambda: net.forward(x_dev, sparse=True))
    g_dense = tm.capture(lambda: net.forward(x_dev, sparse=False))
    tm.region(g_sparse, warmup)
    ms_regions = tm.regions(g_sparse, steps, max(MIN_REGIONS, args.regions), budget_s=25.0)
    ms_step = statistics.median(ms_regions)
    tm.region(g_dense, warmup)
    ms_dense = statistics.median(tm.regions(g_dense, steps, 7, budget_s=8.0))
    flops = stack_flops(batch)
    value = ranks.job_throughput(flops, world, ms_step) / 1e12

    # ---- per-layer device times: a graph of back-to-back launches of one step of the stack on the
    # stack's own buffers (a layer whose tensors fit in L2 runs L2-warm here, as its input does inside
    # the stack, where the layer before has just written it)
    sampler.mark("per_layer")
    iters = args.layer_iters
    per_layer, sums = [], dict(t=0.0, roof=0.0, t_masked=0.0, roof_masked=0.0, flops_masked=0, bytes=0,
                               t_dense_masked=0.0, t_tensor=0.0, roof_tensor=0.0, flops_tensor=0)
    for i, st in enumerate(steps_def):
        res = {}
        for sparse in ((True, False) if st.kind == "conv" else (True,)):
            gr = tm.capture(lambda i=i, sparse=sparse: [net.run_step(i, x_dev, sparse) for _ in range(iters)])
            tm.region(gr, 1)
            res[sparse] = min(tm.region(gr, 2) / 2 for _ in range(3)) / iters
            del gr
        t = res[True]
        if st.kind == "maxpool":
            n, h, w, c = net.outputs[st.src].shape
            bytes_alg = 2 * (net.outputs[st.src].numel() + net.outputs[i].numel())
            f, t_c, t_m, name, bound = 0, 0.0, bytes_alg / (peaks["hbm_gbs"] * 1e9) * 1e3, "maxpool_3x3s2", "hbm"
            row = {"layer": name, "us": round(t * 1e3, 2)}
        else:
            spec = st.spec
            masked = st.kind == "conv"
            f, bytes_alg, t_c, t_m = layer_roofline(spec, peaks, sparse=masked, real_c_in=None if masked else 3)
            if st.res >= 0:
                bytes_alg += 2 * spec.P * spec.C_out
                t_m = bytes_alg / (peaks["hbm_gbs"] * 1e9) * 1e3
            bound = "tensor" if t_c >= t_m else "hbm"
            row = {"layer": spec.name, "us": round(t * 1e3, 2), "tflops": round(f / t / 1e9, 1)}
            if masked:
                row["us_dense"] = round(res[False] * 1e3, 2)
                row["x_dense"] = round(res[False] / t, 3)
                row["plan"] = dict(api.ssconv_plan(net.layers[i]["desc"], True), fold=net.layers[i]["fold"])
                sums["t_masked"] += t
                sums["t_dense_masked"] += res[False]
                sums["roof_masked"] += max(t_c, t_m)
                sums["flops_masked"] += f
                if bound == "tensor":
                    sums["t_tensor"] += t
                    sums["roof_tensor"] += max(t_c, t_m)
                    sums["flops_tensor"] += f
        roof = max(t_c, t_m)
        row.update({"gbs": round(bytes_alg / t / 1e6, 1), "bound": bound, "us_roofline": round(roof * 1e3, 2),
                    "roofline_frac": round(roof / t, 4)})
        per_layer.append(row)
        sums["t"] += t
        sums["roof"] += roof
        sums["bytes"] += bytes_alg

    # ---- end to end with host buffers: every step copies the batch of 3-channel images from pinned
    # host memory, pads them on the device, runs the stack and copies the last activation back.  Copy-in,
    # compute and copy-out run on three streams chained by events, double-buffered on both ends, as a
    # serving loop would do it.
    sampler.mark("e2e")
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    x3_bufs = [torch.empty_like(x_dev) for _ in range(2)]
    torch.cuda.synchronize()
    with torch.cuda.stream(s_run):
        last = net.forward(x_dev, sparse=True)
    torch.cuda.synchronize()
    y_stage = [torch.empty_like(last) for _ in range(2)]
    y_host = [torch.empty(last.shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_run = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(k):
        b = k & 1
        with torch.cuda.stream(s_in):
            if k >= 2:
                s_in.wait_event(ev_run[b])       # step k-2 has read this buffer
            x3_bufs[b].copy_(x3_host, non_blocking=True)
            ev_in[b].record(s_in)
        with torch.cuda.stream(s_run):
            s_run.wait_event(ev_in[b])
            x_dev.copy_(x3_bufs[b], non_blocking=True)   # into the buffer the recorded graph reads (device to device)
            g_sparse.replay()
            if k >= 2:
                s_run.wait_event(ev_out[b])      # the copy-out of step k-2 has read this staging buffer
            y_stage[b].copy_(last, non_blocking=True)
            ev_run[b].record(s_run)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_run[b])
            y_host[b].copy_(y_stage[b], non_blocking=True)
            ev_out[b].record(s_out)

    for k in range(4):
        e2e_step(k)
    torch.cuda.synchronize()
    k_e2e = max(6, min(20, steps))
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tm.barrier()
    t0.record(s_in)
    for k in range(4, 4 + k_e2e):
        e2e_step(k)
    s_out.wait_stream(s_run)
    s_out.wait_stream(s_in)
    t1.record(s_out)
    torch.cuda.synchronize()
    e2e_ms = ranks.max_over_ranks(t0.elapsed_time(t1) / k_e2e, dev)
    h2d, d2h = x3_host.numel() * 2, last.numel() * 2
    e2e_launches = launches
    dev_status = int(net.status.item())
    del net, g_sparse, g_dense, x3_bufs, y_stage
    torch.cuda.empty_cache()

    # ---- the three per-layer sweeps, in short (one GPU only: they are parity-test workloads, reported as context)
    summaries = {}
    if world == 1 and not args.no_summaries:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        for cfg in (2, 3, 4):
            sampler.mark(f"summary_cfg{cfg}")
            m = sweep_measure(cfg, api, synth, torch, tm, dev, peaks, l2_bytes, steps=50, regions=10, layer_iters=50,
                              status=status)
            summaries[f"summary_cfg{cfg}"] = sweep_summary(cfg, m, world, ranks)
            del m
            torch.cuda.empty_cache()
        sampler.mark("summary_e4m3")
        summaries["summary_e4m3"] = fp8_summary(api, synth, torch, tm, dev, l2_bytes, batch, status)
        sampler.mark("summary_convnext_t")
        summaries["summary_convnext_t"] = convnext_summary(api, torch, tm, dev)
        dev_status |= summaries["summary_convnext_t"]["dev_status"]
        dev_status |= int(status.item())
    clocks = sampler.stop() if rank == 0 else None

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import build as oracle_build
        oracle_build.build()
        leg = oracle_leg(15.0)
        cpu = {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample", "images_per_s")}

    if rank == 0:
        sp = spread(ms_regions)
        n_hbm = sum(1 for r in per_layer if r["bound"] == "hbm")
        achieved = flops / (sums["t"] * 1e-3) / 1e12
        ceiling = flops / (sums["roof"] * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD + ("_with_skip_connections" if args.residual else ""),
                       "batch_per_gpu": batch,
                       "stack": "stem 7x7 s2 (dense, on the 3-channel images: space-to-depth + a 4x1 convolution over a "
                                "sliding-window view), 3x3 s2 max-pool, 16 bottlenecks as reduce -> 3x3 -> expand with bias "
                                "+ ReLU, 4 downsample convolutions on their block's input; "
                                + ("skip connections fused into the expand convolutions" if args.residual
                                   else "no residual additions"),
                       "flops": "2*P*C_out*K per convolution (53 of them; the stem with its 3 real channels)",
                       "l2": f"the activations of one step total {act_bytes / 2**30:.1f} GiB (> the {l2_bytes / 2**20:.0f} MiB "
                             f"L2 read from the device): inputs larger than L2",
                       "masks": "magnitude top-2 of 4, selected and compressed once before timing",
                       "launch": "the stack's C-ABI calls recorded into one CUDA graph and replayed",
                       "timing": f"{sp['regions']} regions of {steps} steps, CUDA events on the launching stream, barrier + "
                                 f"synchronize on both sides of each region, max over ranks; ms_per_step is the median",
                       "one_off_prepare_s": round(prep_seconds, 2)},
            "ms_per_step_spread": {k: round(v, 5) if isinstance(v, float) else v for k, v in sp.items()},
            "images_per_s": ranks.job_throughput(batch, world, ms_step),
            "x_dense": ms_dense / ms_step, "ms_per_step_dense": ms_dense,
            "images_per_s_dense": ranks.job_throughput(batch, world, ms_dense),
            "roofline": {
                "bound": "hbm", "kernel": "ssconv_fwd_kernel<sparse> / ssconv_fwd_pair_kernel<sparse> (52 of the 55 steps)",
                "achieved": achieved, "peak": ceiling, "unit": "TFLOP/s", "frac": sums["roof"] / sums["t"],
                "how": "per layer the roofline time is the slower of FLOPs / tensor peak and algorithmic bytes / HBM "
                       "bandwidth; peak = the stack's FLOPs / the sum of those times, achieved = the stack's FLOPs / "
                       "the sum of the measured per-layer CUDA-event times",
                "peak_source": f"{peaks['source']} peaks: HBM {peaks['hbm_gbs']} GB/s; tensor 2 x the dense bf16 burst "
                               f"({peaks['bf16_tflops']} TFLOP/s) for 2:4 layers, 1 x for the dense stem",
                "layers_bound_by": {"hbm": n_hbm, "tensor": len(per_layer) - n_hbm},
                "sum_layer_ms": sums["t"], "sum_roofline_ms": sums["roof"],
                "algorithmic_bytes_per_step": sums["bytes"],
                "achieved_gbs": sums["bytes"] / (sums["t"] * 1e-3) / 1e9, "hbm_peak_gbs": peaks["hbm_gbs"],
                "masked_convolutions": {
                    "sum_layer_ms": sums["t_masked"], "frac": sums["roof_masked"] / sums["t_masked"],
                    "tflops": sums["flops_masked"] / (sums["t_masked"] * 1e-3) / 1e12,
                    "x_dense": sums["t_dense_masked"] / sums["t_masked"]},
                "tensor_bound_layers": {
                    "sum_layer_ms": sums["t_tensor"], "tflops": sums["flops_tensor"] / max(sums["t_tensor"], 1e-9) / 1e9,
                    "peak_tflops": 2.0 * peaks["bf16_tflops"],
                    "frac": sums["roof_tensor"] / max(sums["t_tensor"], 1e-9)},
                "traffic": stack_traffic(batch, args.residual),
                "traffic_note": "dram__bytes_read.sum + dram__bytes_write.sum over the 55 launches of one step (single-pass "
                                "ncu capture at this batch, caches left alone between launches so that write-backs are "
                                "counted in the step; profiles/bench_resnet50_stack_dram_traffic.md); null when the kernel "
                                "sources differ from the ones measured"},
            "per_layer": per_layer,
            "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                    "images_per_s": ranks.job_throughput(batch, world, e2e_ms),
                    "path": "pinned host images [N,224,224,3] bf16 -> device -> the stack -> last activation "
                            "[N,7,7,2048] -> pinned host; three streams, double-buffered"},
            "gpu_launches": len(ms_regions) * steps * launches, "gpu_launches_per_step": launches,
            "gpu_launches_per_e2e_step": e2e_launches,
            "clocks": clocks, "dev_status": dev_status,
        }
        line.update(summaries)
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- per-layer sweep as its own line
def sweep_arm(args):
    """--workload-config 2|3|4: the full line for one of the per-layer sweeps."""
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
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    peaks = load_peaks()
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    tm = Timer(torch, dist, ranks, dev, distributed)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    steps = max(1, min(args.steps, 2000))

    if args.only_layer is not None:   # profiling aid: one layer, launched repeatedly, nothing timed
        spec = (synth.config_layers(5, args.batch or 256) if CONFIG_ID == 5 else timed_layers())[args.only_layer]
        inp = synth.make_inputs(spec)
        desc = api.desc_from_spec(spec)
        w, bias = inp.w.to(dev), inp.bias.to(dev)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        fold = api.ssconv_fold_factor(desc)
        if fold > 1:
            w, bias_f = api.ssconv_fold_weights(desc, fold, w, bias)
            pat, _ = api.ssconv_fold_weights(desc, fold, pat)
            desc, bias = api.ssconv_fold_desc(desc, fold), bias_f
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        n_sets = max(2, -(-int(1.5 * l2_bytes) // (2 * (spec.N * spec.H * spec.W * spec.C_in + spec.P * spec.C_out))) + 1)
        xs = [inp.x.to(dev)] + [torch.randn(inp.x.shape, device=dev).to(torch.bfloat16) for _ in range(n_sets - 1)]
        ys = [torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=dev)
              for _ in range(n_sets)]
        if args.e4m3:   # the same layer on 8-bit operands (2:4 form)
            wq = api.ssconv_quantize_e4m3(w, 16.0)
            pq = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, wq, wq.numel() // 4)
            wq_comp, metaq = api.ssconv_compress_fp8(desc, wq, pq)
            xq = [api.ssconv_quantize_e4m3(x, 1.0) for x in xs]
        if args.pair_tiles is not None:   # the pair kernel with one (0) or two (1) position tiles per work item
            api.ssconv_tune(api.TUNE_PAIR_TILES, args.pair_tiles)
        for i in range(args.layer_iters):
            r = i % n_sets
            if args.e4m3:
                api.ssconv_forward_fp8(desc, xq[r], wq_comp, metaq, bias, 1.0 / 16.0, y=ys[r], dev_status=status)
            elif args.dense:
                api.ssconv_forward_dense(desc, xs[r], w, bias, y=ys[r], dev_status=status)
            else:
                api.ssconv_forward(desc, xs[r], w_comp, meta, bias, y=ys[r], dev_status=status)
        torch.cuda.synchronize()
        if rank == 0:
            sampler.stop()
        print(json.dumps({"only_layer": spec.name, "launches": args.layer_iters, "dense": args.dense,
                          "plan": dict(api.ssconv_plan(desc, not args.dense), fold=fold),
                          "dev_status": int(status.item())}))
        return

    m = sweep_measure(CONFIG_ID, api, synth, torch, tm, dev, peaks, l2_bytes, steps=steps,
                      regions=max(MIN_REGIONS, args.regions), layer_iters=args.layer_iters, status=status, want_e2e=True)
    prep, layers = m["prep"], m["layers"]
    ms_per_step = statistics.median(m["ms_sparse"])
    ms_dense = statistics.median(m["ms_dense"])
    total_flops = m["total_flops"]

    # ---- end to end through the public API with host buffers: every step copies each layer's input
    # from pinned host memory, runs the layer, and copies its output back; three streams chained by events
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
    tm.barrier()
    e2e_t0.record(s_in)
    for _ in range(k_e2e):
        e2e_step(False)
    s_out.wait_stream(s_run)
    s_out.wait_stream(s_in)
    e2e_t1.record(s_out)
    torch.cuda.synchronize()
    e2e_ms = ranks.max_over_ranks(e2e_t0.elapsed_time(e2e_t1) / k_e2e, dev)
    h2d = sum(L["x_host"].numel() * 2 for L in prep)
    d2h = sum(L["y_host"].numel() * 2 for L in prep)
    dev_status = int(status.item())
    clocks = sampler.stop() if rank == 0 else None

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import build as oracle_build
        oracle_build.build()
        leg = oracle_leg(15.0)
        cpu = {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        sparse_peak = 2.0 * peaks["bf16_tflops"]
        achieved = total_flops / (m["sum_kernel_ms"] * 1e-3) / 1e12
        sp = spread(m["ms_sparse"])
        line = {
            "metric": METRIC, "value": ranks.job_throughput(total_flops, world, ms_per_step) / 1e12, "unit": "TFLOP/s",
            "n_gpus": world, "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "layers": len(layers), "batch_per_gpu": layers[0].N,
                       "l2": f"rotating {m['n_sets']} buffer sets of {m['set_bytes'] / 2**20:.0f} MiB (> the "
                             f"{l2_bytes / 2**20:.0f} MiB L2 read from the device) per rank",
                       "masks": "selected and compressed once before timing",
                       "launch": "the C-ABI calls of one step recorded into a CUDA graph per buffer set and replayed",
                       "timing": f"{sp['regions']} regions of {steps} steps; ms_per_step is the median",
                       "one_off_prepare_s": round(m["prep_seconds"], 3)},
            "ms_per_step_spread": {k: round(v, 6) if isinstance(v, float) else v for k, v in sp.items()},
            "x_dense": ms_dense / ms_per_step, "ms_per_step_dense": ms_dense,
            "roofline": {"bound": "tensor", "kernel": "ssconv_fwd_kernel<sparse>", "achieved": achieved,
                         "peak": sparse_peak, "unit": "TFLOP/s", "frac": achieved / sparse_peak,
                         "peak_source": f"2 x dense bf16 burst of {peaks['source']} peaks (nominal sparse:dense ratio)",
                         "layer_mix_ceiling": total_flops / (m["sum_roof_ms"] * 1e-3) / 1e12,
                         "frac_of_layer_mix_ceiling": m["sum_roof_ms"] / m["sum_kernel_ms"],
                         "hbm_peak_gbs": peaks["hbm_gbs"], "traffic": None,
                         "algorithmic_bytes_per_step": m["bytes_alg"]},
            "per_layer": m["per_layer"],
            "e2e": {"value": world * total_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": len(m["ms_sparse"]) * steps * m["launches_per_step"],
            "clocks": clocks, "dev_status": dev_status,
        }
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- entry
def launch_ranks(args, argv):
    """--gpus N > 1 without a torchrun environment: start N ranks of this script, one per GPU."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def main():
    global CONFIG_ID, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="steps per timed region")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--regions", type=int, default=MIN_REGIONS, help="timed regions (at least 30)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-summaries", action="store_true", help="skip the short runs of the three per-layer sweeps")
    ap.add_argument("--layer-iters", type=int, default=None,
                    help="back-to-back launches per layer timing (default 10 for the stack, 100 for the sweeps)")
    ap.add_argument("--only-layer", type=int, default=None,
                    help="a profiling aid: launch just this layer of the chosen configuration (for the stack: the i-th of "
                         "its 52 masked convolutions, on seeded inputs of its own) --layer-iters times and exit")
    ap.add_argument("--dense", action="store_true", help="with --only-layer: use the dense kernel")
    ap.add_argument("--residual", action="store_true",
                    help="fuse the network's skip connections into the expand convolutions of the stack")
    ap.add_argument("--train", action="store_true",
                    help="time one mask-learning step per layer (soft mask, dense forward, weight gradient, "
                         "choice-weight gradient) on one of the per-layer sweeps (default: the ResNet-18 sweep)")
    ap.add_argument("--e4m3", action="store_true", help="with --only-layer: launch the layer's 2:4 e4m3 form")
    ap.add_argument("--pair-tiles", type=int, default=None, choices=[0, 1],
                    help="with --only-layer: force one (0) or two (1) position tiles per work item of the pair kernel")
    ap.add_argument("--convnext", action="store_true",
                    help="only the ConvNeXt-T-shaped forward pass (the default line's summary_convnext_t), one GPU")
    ap.add_argument("--batch", type=int, default=None, help="images per GPU of the stack (default 256)")
    ap.add_argument("--workload-config", type=int, default=None, choices=sorted(WORKLOADS),
                    help="5 (default): the ResNet-50 stack; 2, 3, 4: one of the per-layer sweeps")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_ranks(args, sys.argv[1:]))
    CONFIG_ID = args.workload_config if args.workload_config is not None else (2 if args.train else 5)
    WORKLOAD = WORKLOADS[CONFIG_ID]
    if args.layer_iters is None:
        args.layer_iters = 10 if CONFIG_ID == 5 else 100
    if args.impl == "reference":
        reference_arm(args)
    elif args.convnext:
        convnext_arm(args)
    elif args.train:
        if CONFIG_ID == 5:
            CONFIG_ID, WORKLOAD = 2, WORKLOADS[2]
        train_arm(args)
    elif CONFIG_ID == 5 and args.only_layer is None:
        stack_arm(args)
    else:
        sweep_arm(args)


if __name__ == "__main__":
    main()
