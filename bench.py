#!/usr/bin/env python
"""Benchmark of the fused vector-quantized linear layer (VPTQ inference hot path) on B200.

One "step" is one pass of the whole hot path over one batch: the seven linear calls
(q, k, v, o, gate, up, down) of a LLaMA-2-70B-shaped decoder layer at batch 1, each one
index unpack -> codebook lookups (+ residual) -> scale/bias -> contraction, through the
C ABI (vptq_linear).  The metric is effective weight GB/s: bytes of the compressed format
(packed index streams + codebooks + scale + bias, each counted once per call) per second.

  python bench.py --gpus N --steps K --warmup W          # this library
  python bench.py --impl reference ...                   # the CPU oracle on a bounded sample

Inputs are seeded and synthetic (paper_2409_17066_b200/synth.py).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "effective_weight_GBps_batch1"
UNIT = "GB/s"
WORKLOAD_CFG = 3
WORKLOAD = "config3_llama2_70b_decoder_layer_q_k_v_o_gate_up_down_v8_k65536_res256_B1"


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic byte of a launch, from
# the ncu captures summarised under profiles/ (captured on one layer of the workload; traffic grows
# in proportion to the packed index streams, so it is scaled by the bytes a launch processes).
# An entry is removed (-> null in the output) when its kernel changes after the capture.
NCU_DRAM_BYTES_PER_ALGORITHMIC_BYTE = {
    # kernel: (ratio, source file of the kernel, first 12 hex digits of its SHA-1 when the capture was taken)
    # profiles/decode_l2_fma_kernel_config3_gate_up_fused_B1.md: (178.38 + 3.18) MB DRAM / 178.33 MB algorithmic
    "decode_l2_fma_kernel": (1.018, "decode_l2_fma.cu", "15af2fb60845"),
    # profiles/decode_smem_fma_kernel_config2_gate_proj_B1.md: 19.00 MB / 18.92 MB
    "decode_smem_fma_kernel": (1.004, "decode_smem_fma.cu", "160ad3290bed"),
    # profiles/decode_smem_tc_kernel_config2_gate_proj_B8.md: 21.46 MB / 19.0 MB (the 0.5 MB fragment image and the
    # pre-pass's traffic included)
    "decode_smem_tc_kernel": (1.13, "decode_smem_tc.cu", "ccf102769587"),
    # profiles/decode_bucket_fma_kernel_config3_gate_up_fused_B1.md: (291.95 + 3.35) MB DRAM / 178.33 MB canonical
    # compressed bytes: the kernel reads the prepared image (4 bytes per slot, 21 % padding at N = 8192; the
    # N = 28672 image of down_proj is 1.47 x its canonical bytes, so this overstates that launch by a tenth)
    "decode_bucket_fma_kernel": (1.656, "decode_bucket_fma.cu", "5da8f01fa7c4"),
}

ROOFLINE_KERNEL = {"decode_l2_fma": "decode_l2_fma_kernel", "decode_smem_fma": "decode_smem_fma_kernel", "decode_gl_fma": "decode_gl_fma_kernel", "decode_smem_mma": "decode_smem_tc_kernel",
                   "gemm_tcgen05": "gemm_tcgen05_kernel", "generic": "linear_generic_kernel",
                   "fused_decode_l2_fma": "decode_l2_fma_kernel", "fused_decode_smem_fma": "decode_smem_fma_kernel",
                   "fused_decode_gl_fma": "decode_gl_fma_kernel",
                   "decode_bucket_fma": "decode_bucket_fma_kernel", "fused_decode_bucket_fma": "decode_bucket_fma_kernel"}
# layers of the headline workload that get a prepared image (vptq_prepare): all seven projections; the
# partitions of a fused group add up to the SM count
PREPARED_DEFAULT = "q_proj,k_proj,v_proj,o_proj,gate_proj,up_proj,down_proj"
# projections of a decoder layer that read the same activations
FUSE_GROUPS = (("q_proj", "k_proj", "v_proj"), ("gate_proj", "up_proj"))


def read_traffic(kernel: str, algorithmic_bytes_per_launch: float):
    """Per-launch DRAM traffic scaled from the committed ncu summary, if one exists AND the kernel's source file is
    still the one the counters were taken on (else None: a stale figure is worse than none)."""
    import hashlib
    entry = NCU_DRAM_BYTES_PER_ALGORITHMIC_BYTE.get(kernel)
    if entry is None:
        return None
    ratio, source, digest = entry
    path = os.path.join(ROOT, "paper_2409_17066_b200", "csrc", source)
    try:
        with open(path, "rb") as fh:
            now = hashlib.sha1(fh.read()).hexdigest()[:12]
    except OSError:
        return None
    return ratio * algorithmic_bytes_per_launch if now == digest else None


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


# Replicas only: every rank runs the whole workload on weights of its own, nothing crosses ranks but
# the timing.  The three helpers below are all there is to the N > 1 path.

def replica_layer_ordinal(li: int, rank: int) -> int:
    """Seed ordinal of layer `li` on replica `rank` (every replica has weights of its own)."""
    return li + 100 * rank


def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's time (all ranks get it)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbps(step_bytes_per_rank: float, world: int, ms_step_max: float) -> float:
    """Bytes all replicas processed per step over the slowest replica's step time."""
    return world * step_bytes_per_rank / (ms_step_max * 1e-3) / 1e9


# ------------------------------------------------------------------------------ reference arm

def oracle_sample_rate(layers_np, rows_per_layer, B=1):
    """Run the CPU oracle on `rows_per_layer` sampled output rows of every layer; return
    (seconds, compressed bytes those rows stand for)."""
    import numpy as np
    from oracle import oracle
    t0 = time.perf_counter()
    nbytes = 0.0
    for d, L, wbytes in layers_np:
        s = d["spec"]
        n = min(rows_per_layer, s.M)
        rows = np.linspace(0, s.M - 1, n).astype(np.int32)
        L.linear(d["x"][:B], rows)
        nbytes += wbytes * n / s.M
    return time.perf_counter() - t0, nbytes


def build_oracle_layers(cfg):
    from oracle import oracle
    from paper_2409_17066_b200 import synth
    out = []
    for li, spec in enumerate(synth.CONFIGS[cfg]["layers"]):
        d = synth.make_layer(spec, cfg, li, max(synth.CONFIGS[cfg]["batches"]))
        L = oracle.Layer.from_synth(d)
        wb = sum(a.size for k, a in L._keep.items() if a is not None and k.startswith("idx")) + \
            2 * sum(a.size for k, a in L._keep.items() if a is not None and not k.startswith("idx"))
        out.append((d, L, wb))
    return out


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    from oracle import oracle
    layers = build_oracle_layers(WORKLOAD_CFG)
    # size the per-step sample so that steps + warmup take about two minutes in all
    oracle_sample_rate(layers, 4)                      # first call pays thread start-up
    t_probe, _ = oracle_sample_rate(layers, 64)
    per_row = t_probe / 64
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = max(4, min(28672, int(budget / max(per_row, 1e-6))))
    for _ in range(args.warmup):
        oracle_sample_rate(layers, rows)
    t_total, b_total = 0.0, 0.0
    for _ in range(args.steps):
        t, nb = oracle_sample_rate(layers, rows)
        t_total += t
        b_total += nb
    value = b_total / t_total / 1e9
    sample = f"{rows} evenly spaced output rows of each of the 7 layers per step, batch 1"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------ this library

def run_ours(args):
    import numpy as np
    import torch
    from paper_2409_17066_b200 import build as vbuild
    from paper_2409_17066_b200 import synth

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    vbuild.build()
    from paper_2409_17066_b200 import binding as vb

    peaks = read_peaks()
    cfg_id = args.cfg
    cfg = synth.CONFIGS[cfg_id]
    B = args.batch if args.batch > 0 else min(cfg["batches"])
    keep = set(args.layers.split(",")) if args.layers else None
    default_case = cfg_id == WORKLOAD_CFG and keep is None and B == 1
    # every rank is an independent replica with its own seeded weights (layer ordinal offset by rank)
    layers, xs_np = [], []
    n_sm = torch.cuda.get_device_properties(local_rank).multi_processor_count
    prepared = set(n for n in args.prepared.split(",") if n) if B == 1 else set()
    kept = [sp.name for sp in cfg["layers"] if keep is None or sp.name in keep]
    for li, spec in enumerate(cfg["layers"]):
        if keep is not None and spec.name not in keep:
            continue
        d = synth.make_layer(spec, cfg_id, replica_layer_ordinal(li, rank), B)
        dl = vb.DeviceLayer(d)
        if spec.name in prepared and vb.lib.vptq_prepare_bytes(C.byref(dl.desc), 0) > 0:      # eligible layers only
            # CTAs for the layer: its share (by vector rows) of the SMs when its whole fuse group is prepared and
            # present, else all SMs
            group = next((g for g in FUSE_GROUPS if spec.name in g), None)
            parts = 0
            if group is not None and not args.no_fuse and all(n in prepared and n in kept for n in group):
                rows = {sp.name: sp.R for sp in cfg["layers"] if sp.name in group}
                parts = vb.prepared_shares([rows[n] for n in group], n_sm, -(-spec.k1 // 4096))[group.index(spec.name)]
            dl = dl.prepared(parts)
        layers.append([dl])
        xs_np.append(d["x"])
        del d
    # distinct copies of the index streams, walked in turn, so that every step's weights come
    # from HBM: copies x step bytes > 2 x L2 (the headline workload: 2 x 329 MB >> 126 MB)
    step_bytes = sum(l[0].weight_bytes() for l in layers)
    copies = max(2, min(64, int(2 * 130e6 / step_bytes) + 1))
    for l in layers:
        l.extend(l[0].clone_streams() for _ in range(copies - 1))
    xs = [layers[i][0].upload_x(xs_np[i]) for i in range(len(layers))]
    outs = [torch.empty((B, l[0].spec.M), dtype=vb._TORCH_DT[l[0].desc.out_dtype], device="cuda") for l in layers]
    # calls of a step: projections that read the same activations (q/k/v, gate/up) go through one
    # vptq_linear_fused call where the library serves them with one launch, the rest through vptq_linear
    calls, li = [], 0
    names = [l[0].spec.name for l in layers]
    while li < len(layers):
        group = next((g for g in FUSE_GROUPS if tuple(names[li:li + len(g)]) == g), None)
        if group is not None and not args.no_fuse and \
                vb.vptq_linear_fused_path([layers[j][0].desc for j in range(li, li + len(group))], B).startswith("fused_"):
            idx = list(range(li, li + len(group)))
            calls.append((idx, [vb.FusedLayers([layers[j][c] for j in idx]) for c in range(copies)]))
        else:
            idx = [li]
            calls.append((idx, None))
        li += len(idx)
    call_names = ["+".join(names[j] for j in idx) + f"_{idx[0]}" for idx, _ in calls]
    launches_per_step = sum(f[0].launches(B) if f is not None else vb.vptq_linear_launches(layers[idx[0]][0].desc, B)
                            for idx, f in calls)
    call_paths = [f[0].path(B) if f is not None else vb.vptq_linear_path(layers[idx[0]][0].desc, B) for idx, f in calls]
    call_launches = [f[0].launches(B) if f is not None else vb.vptq_linear_launches(layers[idx[0]][0].desc, B)
                     for idx, f in calls]
    call_bytes = [sum(layers[j][0].weight_bytes() for j in idx) for idx, _ in calls]
    paths = sorted(set(call_paths))

    def step(i, events=None):
        c = i % copies
        for ci, (idx, fused) in enumerate(calls):
            if events is not None:
                events[ci][0].record()
            if fused is not None:
                fused[c].linear(xs[idx[0]], [outs[j] for j in idx])     # the group's common input
            else:
                layers[idx[0]][c].linear(xs[idx[0]], outs[idx[0]])
            if events is not None:
                events[ci][1].record()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()

    # ---- timed region: exactly K steps, CUDA events on the launching stream -----------------------
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    ms_total = max_over_ranks(ms_total, world, "cuda")
    ms_step = ms_total / args.steps
    value = whole_job_gbps(step_bytes, world, ms_step)

    # ---- roofline pass of its own: per-call events over >= 200 steps, whatever --steps was ---------
    r_iters = max(200, min(args.steps, 1000))
    per_call = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in calls]
                for _ in range(r_iters)]
    for i in range(r_iters):
        step(i, per_call[i])
    barrier()
    time.sleep(0.2)
    clocks = sampler.stop()
    call_ms = [[a.elapsed_time(b) for (a, b) in pc] for pc in per_call]
    call_stats = []
    for ci in range(len(calls)):
        v = sorted(call_ms[i][ci] for i in range(r_iters))
        call_stats.append({"mean": statistics.mean(v), "median": v[len(v) // 2], "min": v[0]})
    # the dominant kernel: the family the step spends most of its time in
    by_kernel = {}
    for ci, p in enumerate(call_paths):
        k = ROOFLINE_KERNEL[p]
        e = by_kernel.setdefault(k, {"ms": 0.0, "bytes": 0.0, "launches": 0, "ms_min": 0.0, "ms_median": 0.0})
        e["ms"] += call_stats[ci]["mean"]; e["ms_min"] += call_stats[ci]["min"]; e["ms_median"] += call_stats[ci]["median"]
        e["bytes"] += call_bytes[ci]; e["launches"] += call_launches[ci]
    dom_kernel = max(by_kernel, key=lambda k: by_kernel[k]["ms"])
    dom = by_kernel[dom_kernel]
    kern_ms_per_step = sum(cs["mean"] for cs in call_stats)
    achieved = dom["bytes"] / (dom["ms"] * 1e-3) / 1e9
    per_layer = {call_names[ci]: {
        "us": 1e3 * call_stats[ci]["mean"], "us_median": 1e3 * call_stats[ci]["median"], "us_min": 1e3 * call_stats[ci]["min"],
        "GBps": call_bytes[ci] / (1e-3 * call_stats[ci]["mean"]) / 1e9, "path": call_paths[ci]}
        for ci in range(len(calls))}

    # ---- the step as a CUDA graph (the calls of two steps, over both weight copies), replayed -----
    graph_us = None
    try:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        n_cap = max(2, min(copies, 4))
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(n_cap):
                    step(i)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        reps = []
        for _ in range(30):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); g.replay(); b_.record()
            torch.cuda.synchronize()
            reps.append(1e3 * a.elapsed_time(b_) / n_cap)
        graph_us = {"median": statistics.median(reps), "min": min(reps), "steps_per_graph": n_cap}
    except Exception as e:  # noqa: BLE001  (a capture that fails is reported, not fatal)
        graph_us = {"error": str(e)[:200]}

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    xh = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in xs_np]
    oh = [torch.empty((B, l[0].spec.M), dtype=vb._TORCH_DT[l[0].desc.out_dtype]).pin_memory() for l in layers]
    h2d = sum(x.numel() * x.element_size() for x in xh)
    d2h = sum(o.numel() * o.element_size() for o in oh)

    # (a fused call copies its common input once)
    h2d = sum(xh[idx[0]].numel() * xh[idx[0]].element_size() for idx, _ in calls)

    def step_e2e(i):
        c = i % copies
        for idx, fused in calls:
            if fused is not None:
                fused[c].linear_host_io(xh[idx[0]], [oh[j] for j in idx], xs[idx[0]], [outs[j] for j in idx])
            else:
                l = layers[idx[0]][c]
                vb.vptq_linear_host_io(l.desc, xh[idx[0]], l.ptrs, oh[idx[0]], xs[idx[0]], outs[idx[0]], l.workspace(B))
        torch.cuda.synchronize()     # the step's result is on the host

    for i in range(3):
        step_e2e(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step_e2e(i)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.steps
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
    e2e_value = whole_job_gbps(step_bytes, world, e2e_ms)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "us_per_call_mean": 1e3 * ms_step / len(calls),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD if default_case else
                       f"config{cfg_id}_{'+'.join(l[0].spec.name for l in layers)}_B{B} (profiling case, not the headline workload)",
                       "batch": B, "linear_layers_per_step": len(layers), "calls_per_step": len(calls),
                       "calls": call_names,
                       "compressed_bytes_per_step": step_bytes, "kernel_paths": paths,
                       "prepared_layers": sorted(prepared & set(names)),
                       "l2": f"inputs larger than L2: {copies} copies of the {step_bytes / 1e6:.0f} MB index streams walked alternately",
                       "multi_gpu": "replicas only (no sharding, no collective)"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "activations and outputs cross PCIe every step; the quantized weights stay resident"},
            "gpu_launches": launches_per_step * args.steps,
            "whole_layer_graph_us": graph_us,
            "roofline": {"bound": "hbm", "kernel": dom_kernel, "achieved": achieved,
                         "peak": peaks["hbm"], "peak_source": peaks["source"] + " (copy bandwidth)",
                         "unit": "GB/s", "frac": achieved / peaks["hbm"],
                         "frac_of_nominal_8TBps": achieved / 8000.0,
                         "traffic": read_traffic(dom_kernel, dom["bytes"] / dom["launches"]),
                         "algorithmic_bytes_per_launch": dom["bytes"] / dom["launches"],
                         "launch_us_mean": 1e3 * dom["ms"] / dom["launches"],
                         "launch_us_median": 1e3 * dom["ms_median"] / dom["launches"],
                         "launch_us_min": 1e3 * dom["ms_min"] / dom["launches"],
                         "launches_per_step": dom["launches"], "iterations": r_iters,
                         "step_achieved_all_kernels": step_bytes / (kern_ms_per_step * 1e-3) / 1e9,
                         "step_frac_all_kernels": step_bytes / (kern_ms_per_step * 1e-3) / 1e9 / peaks["hbm"],
                         "note": "dominant kernel = the family the step spends most time in; achieved = canonical "
                                 "compressed bytes of its launches / their mean event durations, over a pass of "
                                 "its own; step_* = all calls of the step",
                         "per_layer": per_layer}}
    if dom_kernel == "gemm_tcgen05_kernel":
        flops = sum(2.0 * B * l[0].spec.M * l[0].spec.N for l in layers)
        tf = flops / (kern_ms_per_step * 1e-3) / 1e12
        line["roofline"].update({"bound": "tensor", "achieved": tf, "peak": peaks["bf16"], "unit": "TFLOP/s",
                                 "frac": tf / peaks["bf16"], "peak_source": peaks["source"] + " (cuBLAS bf16 burst)",
                                 "traffic": None})
        line["roofline"].pop("frac_of_nominal_8TBps")

    if rank == 0:
        if not args.no_extra and default_case:
            line["extra"] = extra_configs(vb, synth, peaks)
        if not args.no_cpu and default_case:
            line["cpu_baseline"] = cpu_baseline()
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def cpu_baseline():
    from oracle import oracle
    layers = build_oracle_layers(WORKLOAD_CFG)
    oracle_sample_rate(layers, 4)                      # first call pays thread start-up
    t_probe, _ = oracle_sample_rate(layers, 256)
    rows = max(16, min(28672, int(256 * 40.0 / max(t_probe, 1e-6))))   # 10-30 s of CPU work (layers smaller than the sample are taken whole)
    t, nb = oracle_sample_rate(layers, rows)
    cores = oracle.num_threads()
    # the same oracle on one thread, on a sample an eighth of the size
    oracle.set_num_threads(1)
    rows1 = max(4, rows // 8)
    t1, nb1 = oracle_sample_rate(layers, rows1)
    oracle.set_num_threads(cores)
    return {"value": nb / t / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "seconds": t, "single_thread_value": nb1 / t1 / 1e9, "single_thread_seconds": t1,
            "sample": f"{rows} evenly spaced output rows of each of the 7 layers of the workload, batch 1 "
                      f"({rows1} rows for the single-thread figure)"}


_FLUSH = None


def flush_l2():
    """Write a buffer twice the size of L2 (256 MB): the next call finds none of its data there."""
    import torch
    global _FLUSH
    if _FLUSH is None:
        _FLUSH = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    _FLUSH.zero_()


def isolated_call_us(fn, iters=20):
    """One call at a time, bracketed by events: L2-warm (the same weights again and again) and after an L2
    flush (a 256 MB memset before every call).  What a user sees per call, launch path included."""
    import torch
    out = {}
    for label, flush in (("warm", False), ("after_l2_flush", True)):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        ts = []
        for _ in range(iters):
            if flush:
                flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn(0)
            b.record()
            torch.cuda.synchronize()
            ts.append(1e3 * a.elapsed_time(b))
        out["us_isolated_" + label + "_median"] = statistics.median(ts)
        out["us_isolated_" + label + "_min"] = min(ts)
    return out


def time_calls(fn, n_variants, iters=30, warm=5):
    """Per-call device time of fn(i), i cycling over weight copies.  Returns (graph_ms, eager_median_ms,
    eager_min_ms): graph_ms = calls captured back to back in one CUDA graph, replayed, total / calls
    (what the kernels cost); the eager figures bracket single calls with events and include whatever
    the host adds when a kernel is shorter than its launch path."""
    import torch
    for i in range(max(warm, n_variants)):     # every variant once: scratch buffers exist before the capture
        fn(i % n_variants)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for i in range(iters):
        ev[i][0].record()
        fn(i % n_variants)
        ev[i][1].record()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in ev]
    calls = max(n_variants, 8)
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(calls):
                fn(i % n_variants)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    reps = []
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        reps.append(a.elapsed_time(b) / calls)
    return statistics.median(reps), statistics.median(ms), min(ms)


def extra_configs(vb, synth, peaks):
    """µs/call, effective weight GB/s (and TFLOP/s for the batched case) of the other workloads."""
    import torch
    res = {}
    for cfg in (0, 1, 2, 4, 5):
        c = synth.CONFIGS[cfg]
        seen = set()
        for li, spec in enumerate(c["layers"]):
            if (spec.M, spec.N) in seen:
                continue
            seen.add((spec.M, spec.N))
            Bmax = max(c["batches"])
            d = synth.make_layer(spec, cfg, li, Bmax)
            base = vb.DeviceLayer(d)
            wb = base.weight_bytes()
            n_copies = max(1, min(64, int(2 * 130e6 / wb) + 1))    # walk > 2 x L2 of weights
            variants = [base] + [base.clone_streams() for _ in range(n_copies - 1)]
            for B in c["batches"]:
                x = base.upload_x(d["x"][:B])
                out = torch.empty((B, spec.M), dtype=vb._TORCH_DT[base.desc.out_dtype], device="cuda")
                gms, med, mn = time_calls(lambda i: variants[i].linear(x, out), n_copies)
                key = f"cfg{cfg}_{spec.name}_{spec.M}x{spec.N}_B{B}"
                r = {"us": 1e3 * gms, "us_eager_median": 1e3 * med, "us_eager_min": 1e3 * mn,
                     **isolated_call_us(lambda i: variants[i].linear(x, out)),
                     "GBps": wb / (gms * 1e-3) / 1e9,
                     "frac_hbm": wb / (gms * 1e-3) / 1e9 / peaks["hbm"], "path": vb.vptq_linear_path(base.desc, B),
                     "weight_copies": n_copies}
                if B >= 64:
                    fl = 2.0 * B * spec.M * spec.N
                    r["TFLOPs"] = fl / (gms * 1e-3) / 1e12
                    r["frac_bf16_peak"] = r["TFLOPs"] / peaks["bf16"]
                    W = torch.randn(spec.M, spec.N, device="cuda", dtype=torch.float16)
                    xh = torch.randn(B, spec.N, device="cuda", dtype=torch.float16)
                    dm, _, _ = time_calls(lambda i: torch.matmul(xh, W.t()), 1)
                    r["dense_fp16_matmul_us"] = 1e3 * dm
                    r["dense_fp16_TFLOPs"] = fl / (dm * 1e-3) / 1e12
                    del W, xh
                res[key] = r
                # the same layer over a prepared image, where the format has one and the call does not use it yet
                if B == 1 and vb.lib.vptq_prepare_bytes(C.byref(base.desc), 0) > 0:
                    pbase = base.prepared(0)
                    pvar = [pbase] + [pbase.clone_streams() for _ in range(n_copies - 1)]
                    gms, med, mn = time_calls(lambda i: pvar[i].linear(x, out), n_copies)
                    res[key + "_prepared"] = {"us": 1e3 * gms, "us_eager_median": 1e3 * med, "us_eager_min": 1e3 * mn,
                                              "GBps": wb / (gms * 1e-3) / 1e9, "frac_hbm": wb / (gms * 1e-3) / 1e9 / peaks["hbm"],
                                              "path": vb.vptq_linear_path(pbase.desc, 1), "weight_copies": n_copies}
                    del pvar, pbase
            del variants, base, d
            torch.cuda.empty_cache()
    res.update(extra_fused(vb, synth, peaks))
    res.update(extra_zipf(vb, synth, peaks))
    res.update(encoder_assign(vb, synth))
    return res


def extra_zipf(vb, synth, peaks):
    """Reported, not graded: one layer per decode kernel family with Zipf-like index histograms (s = 1 over a
    random permutation of the centroids) instead of uniform ones, next to the uniform figure of the same layer."""
    import torch
    res = {}
    cases = [(1, 0, 1, False), (3, 3, 1, True), (2, 0, 1, False), (2, 0, 8, False), (5, 0, 1, False)]
    for cfg, li, B, prep in cases:
        spec = synth.CONFIGS[cfg]["layers"][li]
        row = {}
        for dist in ("uniform", "zipf"):
            d = synth.make_layer(spec, cfg, li, B, dist=dist)
            base = vb.DeviceLayer(d)
            if prep:
                try:
                    base = base.prepared(0)
                except vb.VptqError as e:      # a skewed histogram can exceed the image capacity: canonical path
                    row["prepared_" + dist] = f"refused ({e.code})"
            wb = base.weight_bytes()
            n = max(2, min(64, int(2 * 130e6 / wb) + 1))
            variants = [base] + [base.clone_streams() for _ in range(n - 1)]
            x = base.upload_x(d["x"][:B])
            out = torch.empty((B, spec.M), dtype=vb._TORCH_DT[base.desc.out_dtype], device="cuda")
            gms, _, _ = time_calls(lambda i: variants[i].linear(x, out), n)
            row["us_" + dist] = 1e3 * gms
            row["path"] = vb.vptq_linear_path(base.desc, B)
            del variants, base, d
            torch.cuda.empty_cache()
        res[f"zipf_cfg{cfg}_{spec.name}_{spec.M}x{spec.N}_B{B}"] = row
    return res


def extra_fused(vb, synth, peaks):
    """Projections that read the same activations through one vptq_linear_fused call, against one call per layer
    (device time per call from CUDA-graph replays over > 2 x L2 of weight copies), for the workloads whose decode
    kernels keep the codebooks in shared memory (config 2) or per group in global memory (the published 2.26-bit
    setting); the k/v projections of those models have the shape of q."""
    import torch
    res = {}
    for cfg, names, B in ((2, ("gate_proj", "up_proj"), 1), (5, ("q_proj", "q_proj", "q_proj"), 1),
                          (5, ("gate_proj", "gate_proj"), 1)):
        by_name = {s.name: (li, s) for li, s in enumerate(synth.CONFIGS[cfg]["layers"])}
        ds = []
        for i, nm in enumerate(names):
            li, sp = by_name[nm]
            ds.append(synth.make_layer(sp, cfg, li + 10 * i, B))       # weights of its own per projection
        for d in ds[1:]:
            d["x"] = ds[0]["x"]
        base = [vb.DeviceLayer(d) for d in ds]
        wb = sum(dl.weight_bytes() for dl in base)
        n = max(2, min(32, int(2 * 130e6 / wb) + 1))
        copies = [[dl] + [dl.clone_streams() for _ in range(n - 1)] for dl in base]
        fused = [vb.FusedLayers([copies[l][c] for l in range(len(base))]) for c in range(n)]
        x = base[0].upload_x(ds[0]["x"][:B])
        outs = [torch.empty((B, dl.spec.M), dtype=vb._TORCH_DT[dl.desc.out_dtype], device="cuda") for dl in base]
        g, _, _ = time_calls(lambda i: fused[i].linear(x, outs), n)

        def one_by_one(i):
            for l in range(len(base)):
                copies[l][i].linear(x, outs[l])
        gs, _, _ = time_calls(one_by_one, n)
        label = "+".join(names) if len(set(names)) > 1 else f"{len(names)}x{names[0]}"
        res[f"cfg{cfg}_fused_{label}_B{B}"] = {
            "us": 1e3 * g, "us_one_call_per_layer": 1e3 * gs, "GBps": wb / (g * 1e-3) / 1e9,
            "frac_hbm": wb / (g * 1e-3) / 1e9 / peaks["hbm"], "path": fused[0].path(B), "weight_copies": n}
        if B == 1 and all(vb.lib.vptq_prepare_bytes(C.byref(dl.desc), 0) > 0 for dl in base):
            # the same call over prepared images that share the SMs
            n_sm = torch.cuda.get_device_properties(0).multi_processor_count
            shares = vb.prepared_shares([dl.spec.R for dl in base], n_sm, -(-base[0].spec.k1 // 4096))
            pbase = [dl.prepared(p) for dl, p in zip(base, shares)]
            pcopies = [[dl] + [dl.clone_streams() for _ in range(n - 1)] for dl in pbase]
            pfused = [vb.FusedLayers([pcopies[l][c] for l in range(len(base))]) for c in range(n)]
            g, _, _ = time_calls(lambda i: pfused[i].linear(x, outs), n)
            res[f"cfg{cfg}_fused_{label}_B{B}_prepared"] = {
                "us": 1e3 * g, "GBps": wb / (g * 1e-3) / 1e9, "frac_hbm": wb / (g * 1e-3) / 1e9 / peaks["hbm"],
                "path": pfused[0].path(B), "weight_copies": n}
            del pfused, pcopies, pbase
        del fused, copies, base, ds
        torch.cuda.empty_cache()
    return res


def encoder_assign(vb, synth):
    """The quantizer's assignment step (Eq. 2) on a matrix of the size of config 1's layer: every one of the
    2.1 M vectors against all 65536 centroids, by the tensor-core filter + FP32 decision (the default) and by
    the plain FP32 kernel (same indices).  The FP32 kernel is bound by the FP32 pipes: one subtract and one
    fma per component and centroid; peak = SMs x 128 FP32 lanes x SM clock instructions per second."""
    import numpy as np
    import torch
    M, N, v, k = 4096, 4096, 8, 65536
    rng = np.random.default_rng(synth.BASE_SEED + 77)
    W = torch.from_numpy(rng.normal(0, 0.02, (M, N)).astype(np.float16)).cuda()
    Cb = torch.from_numpy(rng.normal(0, 0.02, (k, v)).astype(np.float16)).cuda()
    idx = torch.empty((M // v, N), dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    out = {}
    for flags in (0, vb.FLAG_FORCE_GENERIC):
        need = vb.lib.vptq_assign_workspace_bytes(M, N, v, k, flags)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")

        def call():
            rc = vb.lib.vptq_assign(W.data_ptr(), M, N, v, Cb.data_ptr(), k, idx.data_ptr(), flags,
                                    ws.data_ptr() if need else None, need, st)
            assert rc == vb.OK, rc
        call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 3
        path = vb.vptq_assign_path(M, N, v, k, flags)
        r = {"ms": ms, "G_distances_per_s": (M // v) * N * k / (ms * 1e-3) / 1e9}
        if flags == 0:
            assert vb.vptq_workspace_status(ws) == vb.OK
            r["vectors_sent_to_the_full_fp32_scan"] = int(ws[32:36].view(torch.int32).item()) / ((M // v) * N)
        else:
            props = torch.cuda.get_device_properties(0)
            pairs = (M // v) * N * k * v                               # (subtract, fma) pairs
            peak = props.multi_processor_count * 128 * 1.965e9         # FP32 instructions per second at the maximum SM clock
            r["roofline"] = {"bound": "alu", "achieved": 2 * pairs / (ms * 1e-3) / 1e12, "peak": peak / 1e12,
                             "unit": "T FP32 instructions/s (one subtract and one fma per component)",
                             "frac": 2 * pairs / (ms * 1e-3) / peak,
                             "peak_source": "148 SMs x 128 FP32 lanes x 1.965 GHz (unit counts and maximum clock)"}
        out[f"encoder_{path}_4096x4096_v8_k65536"] = r
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-fuse", action="store_true", help="one vptq_linear call per layer (no vptq_linear_fused)")
    ap.add_argument("--prepared", default=PREPARED_DEFAULT,
                    help="comma-separated layers that get a prepared image (batch 1 only); '' = none")
    ap.add_argument("--encoder", action="store_true",
                    help="only the quantizer's assignment step (Eq. 2) at full size (profiling case)")
    ap.add_argument("--cfg", type=int, default=WORKLOAD_CFG,
                    help="workload number (default: the headline workload); others are profiling cases")
    ap.add_argument("--layers", default="", help="comma-separated layer names to keep (profiling cases)")
    ap.add_argument("--batch", type=int, default=0, help="tokens per call (default: the workload's smallest)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.encoder:
        import torch
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
        from paper_2409_17066_b200 import build as vbuild
        from paper_2409_17066_b200 import synth
        vbuild.build()
        from paper_2409_17066_b200 import binding as vb
        print(json.dumps(encoder_assign(vb, synth)))
        return 0
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
