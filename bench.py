#!/usr/bin/env python
"""Benchmark of the ResIST hot path on B200: sub-ResNet training images/s.

Workload (N = 1, default `--workload wide`): the wide CIFAR-shaped bottleneck ResNet [3,4,23,3] (64..512 x4 channels,
32x32x3 inputs, 100 classes): S = 8 sub-ResNets from a seeded layer-wise partition (the non-first blocks of the third
section are dealt out), batch 128 per sub-ResNet, bf16 activations and weights with fp32 master weights, 50 local SGD
steps per synchronisation round.  It is the largest training configuration by work per step (7 TFLOP) and every layer
of it is tensor-core shaped.  `--workload resnet110` and `--workload imagenet` time the other two training
configurations the same way, `--workload reassembly` the synchronisation kernels alone.
A "step" is one grouped local step of all S sub-ResNets (S*B images: forward, backward, SGD-momentum update); every
50th step (the counter runs on through warm-up and repeats) is followed by the reassembly (resist_aggregate) and the
next round's partition + scatter (resist_partition) inside the timed region.  A block of exactly K steps is timed
with CUDA events, blocks are repeated until about 1.5 s is measured, and the median block is reported with its spread.
Inputs are synthetic (Gaussian pixels, uniform labels), generated before the timed region.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload wide|resnet110|imagenet|reassembly]

`value` is measured with the inputs resident in HBM; `e2e` repeats the same steps through the same public calls
with the inputs in pinned host memory: every step's inputs are copied to the device inside the timed region (on a copy
stream, into one of two staging sets, so that the copy for the next step runs beside the current step) and every
step's losses are copied back to pinned host memory.
With --gpus N > 1 (under torchrun) every rank runs an independent replica on its own GPU and the values add up:
the path has no exchange between GPUs.
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

import synth  # noqa: E402

# workload name -> (synth configuration number, description, distinct batches per sub-ResNet that are cycled)
WORKLOADS = {
    "wide": (3, "configs[2]: wide CIFAR-shaped bottleneck ResNet [3,4,23,3] (64..512 x4), 32x32x3, 100 classes, S=8 sub-ResNets, "
                "batch 128 per sub-ResNet, bf16 + fp32 master, 50 local steps per round", 8),
    "resnet110": (2, "configs[1]: CIFAR-shaped ResNet-110, S=4 sub-ResNets, batch 128 per sub-ResNet, bf16 + fp32 master, "
                     "50 local steps per round", 16),
    "imagenet": (4, "configs[3]: ImageNet-shaped ResNet-101, 224x224x3, 1000 classes, S=4 sub-ResNets, batch 64 per sub-ResNet, "
                    "bf16 + fp32 master, 20 local steps per round", 3),
    # the paper's local-SGD baseline (Sec. 2.4) on the same kernels: no block is dealt out, every sub-ResNet is the full network
    "wide_localsgd": (3, "configs[2]'s network trained by local SGD (Sec. 2.4): no block dealt out, S=8 full replicas, batch 128 each, "
                         "bf16 + fp32 master, 50 local steps per round", 4),
}
# DRAM traffic of a kernel family as a fraction of its algorithmic bytes (dram__bytes_read.sum + dram__bytes_write.sum over the
# family's launches of one step / the library's byte count of the same launches), from the ncu capture summarised in
# profiles/dram_traffic_conv_tc_kernel_wide_S2_B128.txt: workload -> family -> ratio.  The capture ran 2 of the 8 sub-ResNets (the
# full workload is too large to capture); the full launch's traffic is reported as ratio x its algorithmic bytes, a lower bound,
# since with 8 sub-ResNets less of each tensor is still in L2 when its consumer reads it.
NCU_TRAFFIC_RATIO = {"wide": {"conv_fwd_tcgen05": 0.716, "conv_fwd_tcgen05@tensor": 0.581, "conv_dgrad_tcgen05": 0.576,
                              "conv_dgrad_tcgen05@tensor": 0.531}}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU, sampled every 200 ms while running."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(ms: float, device) -> float:
    """The slowest rank's time: with N independent replicas the job's throughput is the images of all ranks over it."""
    import torch
    import torch.distributed as dist
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def make_batches(cfg, n):
    xs, ys = [], []
    for i in range(n):
        bx, by = [], []
        for s in range(cfg.S):
            x, y = synth.batch(cfg, 0, i, s)
            bx.append(x)
            by.append(y)
        xs.append(bx)
        ys.append(by)
    return xs, ys


def workload_config(args):
    cfg = synth.config(WORKLOADS[args.workload][0])
    if args.workload == "wide_localsgd":
        cfg.arch = synth.wide_cifar_arch(policy="none")
    # a smaller case of the same kernels for profiler captures (a few GB on the device): fewer sub-ResNets, smaller batch
    if args.subnets:
        cfg.S = args.subnets
    if args.batch:
        cfg.batch = args.batch
    return cfg


def bound_of(name: str, v: dict, peaks: dict) -> dict:
    """Roofline of one profile entry: entries named '<family>@tensor' hold the launches whose arithmetic intensity is above the
    ridge (held against the sustained bf16 peak, the kernels being timed inside a long step), the others against HBM bandwidth."""
    ms = max(v["ms"], 1e-9)
    if name.endswith("@tensor"):
        ach, peak, unit, bound = v["flops"] / ms / 1e9, peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"], "TFLOP/s", "tensor"
    else:
        ach, peak, unit, bound = v["bytes"] / ms / 1e6, peaks["hbm_gbs"], "GB/s", "hbm"
    return {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak}


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2107_00961_b200 as lib

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    cfg = workload_config(args)
    S, B, K, W = cfg.S, cfg.batch, args.steps, args.warmup
    LOCAL_STEPS = cfg.local_steps
    POOL = WORKLOADS[args.workload][2]
    a = cfg.arch

    ctx = lib.Context(a.to_int32(), dtype=lib.BF16, momentum=cfg.momentum, seed=cfg.init_seed, device=str(dev))
    p0, b0 = synth.init_params(a, cfg.init_seed)
    ctx.set_params(p0, b0)
    xs, ys = make_batches(cfg, POOL)
    d_x = [[torch.from_numpy(x).to(dev).to(torch.bfloat16) for x in bx] for bx in xs]
    d_y = [[torch.from_numpy(y).to(dev) for y in by] for by in ys]
    h_x = [[torch.from_numpy(synth.bf16_bits(x).view(np.int16)).view(torch.bfloat16).pin_memory() for x in bx] for bx in xs]
    h_y = [[torch.from_numpy(y).pin_memory() for y in by] for by in ys]
    # end-to-end pass: two sets of device staging buffers; the copy of step i+1's inputs (pinned host memory -> device, on a
    # copy stream) runs while step i computes, and every step's losses are copied to their own slot of a pinned host ring
    stage_x = [[torch.empty_like(d_x[0][s]) for s in range(S)] for _ in range(2)]
    stage_y = [[torch.empty_like(d_y[0][s]) for s in range(S)] for _ in range(2)]
    loss = torch.zeros(S, dtype=torch.float32, device=dev)
    h_loss = torch.zeros(256, S, dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream(device=dev)
    ev_copied = [torch.cuda.Event() for _ in range(2)]
    ev_free = [torch.cuda.Event() for _ in range(2)]
    for e in ev_free:
        e.record(stream)
    state = {"step": 0, "round": 0, "launches": 0, "boundaries": 0}

    def new_round():
        ctx.partition(cfg.round_seed(state["round"]), S)
        state["round"] += 1

    def one_step(e2e: bool):
        i = state["step"] % POOL
        if e2e:
            b = state["step"] % 2
            copy_stream.wait_event(ev_free[b])                    # the step that last used this staging set has finished
            with torch.cuda.stream(copy_stream):
                for s in range(S):
                    stage_x[b][s].copy_(h_x[i][s], non_blocking=True)
                    stage_y[b][s].copy_(h_y[i][s], non_blocking=True)
                ev_copied[b].record(copy_stream)
            stream.wait_event(ev_copied[b])
            ctx.local_step_grouped(stage_x[b], stage_y[b], cfg.lr, loss)
            h_loss[state["step"] % h_loss.shape[0]].copy_(loss, non_blocking=True)   # this step's losses, read by the host after the run
            ev_free[b].record(stream)
        else:
            ctx.local_step_grouped(d_x[i], d_y[i], cfg.lr, loss)
        state["step"] += 1                    # the step counter runs on through warm-up and all repeats: round boundaries fall where they fall
        state["launches"] += ctx.step_info()["kernel_launches"]
        if state["step"] % LOCAL_STEPS == 0:
            ctx.aggregate()
            new_round()
            state["launches"] += 3            # aggregate (one launch) + scatter (parameters, buffers)
            state["boundaries"] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(e2e: bool):
        """W warm-up steps, then blocks of exactly K steps, each bracketed by a barrier and CUDA events, repeated until about 1.5 s of
        device time has been measured (at least 3 blocks): the reported time is the median block, the spread is kept."""
        state.update(step=0, round=0)         # both passes train the same sequence of partitions (a partition's shape sets the step time)
        new_round()
        for _ in range(W):
            one_step(e2e)
        blocks, launches, bounds = [], [], []
        total = 0.0
        while len(blocks) < (1 if args.profile_case else 3) or (not args.profile_case and total < 1500.0 and len(blocks) < 200):
            state.update(launches=0, boundaries=0)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(K):
                one_step(e2e)
            e1.record(stream)
            barrier()
            ms = max_over_ranks(e0.elapsed_time(e1), dev)
            blocks.append(ms); launches.append(state["launches"]); bounds.append(state["boundaries"])
            total += ms
        return blocks, launches, bounds

    sampler = ClockSampler(local)
    sampler.start()
    blocks, launches, bounds = timed(False)
    clocks = sampler.stop()
    info = ctx.step_info()
    if args.profile_case:                  # profiler capture: the resident pass alone, then a few profiled steps
        print(json.dumps({"profile_case": True, "workload": args.workload, "S": S, "batch_per_subnet": B, "ms_per_step": float(np.median(blocks)) / K}))
        return
    blocks_e2e, _, _ = timed(True)
    assert bool(torch.isfinite(h_loss).all()), "the end-to-end pass produced a non-finite loss"
    ms = float(np.median(blocks))
    ms_e2e = float(np.median(blocks_e2e))
    mid = int(np.argsort(blocks)[len(blocks) // 2])

    # round boundary alone: reassembly + next partition (scatter, new launch plan) after a step, CUDA events around the two calls
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    over = []
    for _ in range(3):
        one_step(False)
        torch.cuda.synchronize()
        e0.record(stream)
        ctx.aggregate()
        new_round()
        ctx.local_step_grouped(d_x[0], d_y[0], cfg.lr, loss)     # the first step of a round builds the round's launch plan
        e1.record(stream)
        torch.cuda.synchronize()
        over.append(e0.elapsed_time(e1))
    round_overhead_ms = float(np.median(over)) - ms / K

    # per-kernel pass: the same steps with every launch bracketed by CUDA events on the library's stream
    peaks = measured_peaks()
    ctx.set_profiling(True)
    ctx.get_profile()
    state.update(step=0, round=0)
    new_round()
    nprof = min(max(K, 4), 10)
    for _ in range(nprof):
        one_step(False)
    prof = ctx.get_profile()
    # the reassembly kernels on this workload's parameter set (they run once per round: timed here in a loop of their own)
    for i in range(10):
        ctx.aggregate()
        ctx.partition(cfg.round_seed(100 + i), S)
    sync_prof = ctx.get_profile()
    ctx.set_profiling(False)
    step_prof = {k: v for k, v in prof.items() if k not in ("scatter", "aggregate")}
    total_ms = sum(v["ms"] for v in step_prof.values())
    families = {}
    for k, v in sorted(step_prof.items(), key=lambda kv: -kv[1]["ms"]):
        r = bound_of(k, v, peaks)
        families[k] = {"ms_per_step": v["ms"] / nprof, "share": v["ms"] / total_ms, "launches_per_step": v["operations"] / nprof, **r}
    top_name, top = max(step_prof.items(), key=lambda kv: kv[1]["ms"])
    roof = {"kernel": top_name, "share_of_step": top["ms"] / total_ms, "launches": top["operations"], "avg_ms": top["ms"] / top["operations"],
            **bound_of(top_name, top, peaks), "peak_source": peaks["source"] + " (MEASURED_PEAKS.json)" if peaks["source"] == "measured" else "fallback",
            "algorithmic_bytes_per_launch": top["bytes"] / top["operations"], "algorithmic_flops_per_launch": top["flops"] / top["operations"],
            "arithmetic_intensity": top["flops"] / max(top["bytes"], 1.0),
            # DRAM bytes (read + written) per launch of that family from the ncu capture summarised under profiles/; None for a
            # family the capture does not cover or whose kernel has changed since
            "traffic": (NCU_TRAFFIC_RATIO.get(args.workload, {}).get(top_name) or 0.0) * top["bytes"] / top["operations"] or None}
    if roof["traffic"]:
        roof["traffic_source"] = "ncu on 2 of the 8 sub-ResNets, scaled by algorithmic bytes (lower bound: see profiles/dram_traffic_conv_tc_kernel_wide_S2_B128.txt)"
    conv = {k: v for k, v in step_prof.items() if k.startswith("conv_")}
    conv_ms = sum(v["ms"] for v in conv.values()) + sum(v["ms"] for k, v in step_prof.items() if k.startswith("wgrad_splitk"))
    conv_flops = sum(v["flops"] for v in conv.values())
    tens = {k: v for k, v in conv.items() if k.endswith("@tensor")}
    tens_ms, tens_flops = sum(v["ms"] for v in tens.values()), sum(v["flops"] for v in tens.values())
    reassembly = {}
    for name in ("scatter", "aggregate"):
        if name in sync_prof:
            v = sync_prof[name]
            gbps = v["bytes"] / max(v["ms"], 1e-9) / 1e6
            reassembly[name] = {"us_per_call": v["ms"] / v["operations"] * 1e3, "MB_per_call": v["bytes"] / v["operations"] / 1e6, "GBps": gbps,
                                "frac_of_hbm_peak": gbps / peaks["hbm_gbs"]}

    images = S * B * K * world
    out = {
        "metric": "sub-ResNet train images/s", "value": images / (ms * 1e-3), "unit": "images/s", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload][1] + "; every %d-th step is followed by resist_aggregate + resist_partition inside the timed region" % LOCAL_STEPS,
                   "S": S, "batch_per_subnet": B, "local_steps": LOCAL_STEPS, "multi_gpu": "independent replicas" if world > 1 else "single GPU",
                   "l2": "working set per step (saved activations, %.0f MB) exceeds the 126 MB L2; no flush" % (info["workspace_bytes"] / 1e6)},
        "timing": {"blocks": len(blocks), "steps_per_block": K, "ms_per_step_min": min(blocks) / K, "ms_per_step_max": max(blocks) / K,
                   "round_boundaries_in_timed_blocks": int(sum(bounds)), "round_boundaries_in_median_block": int(bounds[mid]),
                   "round_overhead_ms": round_overhead_ms,
                   "ms_per_step_amortised_over_a_round": ms / K if sum(bounds) else (ms / K * LOCAL_STEPS + round_overhead_ms) / LOCAL_STEPS,
                   "note": "value = median block of exactly K steps; round_overhead_ms = aggregate + partition + plan rebuild of one round boundary, timed alone"},
        "clocks": clocks,
        "e2e": {"value": images / (ms_e2e * 1e-3), "unit": "images/s", "ms_per_step": ms_e2e / K,
                "h2d_bytes_per_step": int(S * (B * a.in_h * a.in_w * a.in_c * 2 + B * 4)), "d2h_bytes_per_step": int(S * 4)},
        "gpu_launches": int(launches[mid]),
        "conv": {"TFLOPs": conv_flops / max(conv_ms, 1e-9) / 1e9, "frac_of_bf16_peak": conv_flops / max(conv_ms, 1e-9) / 1e9 / peaks["bf16_tflops"],
                 "tensor_bound_TFLOPs": tens_flops / max(tens_ms, 1e-9) / 1e9,
                 "tensor_bound_frac_of_sustained_bf16_peak": tens_flops / max(tens_ms, 1e-9) / 1e9 / (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"]),
                 "tensor_bound_share_of_conv_flops": tens_flops / max(conv_flops, 1.0),
                 "tensor_core_convs": info["tensor_core_convs"], "cuda_core_convs": info["cuda_core_convs"],
                 "flops_per_step": info["conv_flops"]},
        "roofline": roof, "families": families, "reassembly": reassembly,
    }
    if rank == 0:
        if not args.skip_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(cfg, budget_s=20.0)
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def oracle_step_all(cfg, a, mask, params, B, step_idx, subs=None):
    """One oracle local step of the sub-ResNets in `subs` (default all) at batch B, one thread per sub-ResNet.  Returns seconds."""
    import oracle
    subs = list(range(cfg.S)) if subs is None else subs
    data = {s: synth.batch(cfg, 0, step_idx, s, B=B, as_bf16=True) for s in subs}
    moms = {s: np.zeros_like(params[s]) for s in subs}
    t0 = time.perf_counter()
    th = [threading.Thread(target=oracle.step, args=(a, oracle.present_of(mask, s), params[s], moms[s], None, data[s][0], data[s][1]),
                           kwargs=dict(lr=cfg.lr, mu=cfg.momentum, quant=0)) for s in subs]
    for t in th:
        t.start()
    for t in th:
        t.join()
    return time.perf_counter() - t0


def cpu_sample(cfg):
    """Sub-ResNets per oracle step: as many as the host has cores, at most S (one thread each)."""
    return list(range(min(cfg.S, max(1, os.cpu_count() or 1))))


def cpu_baseline(cfg, budget_s: float):
    """The oracle as it stands, on the host cores: one local step at a reduced batch, one thread per sub-ResNet."""
    import oracle
    a = cfg.arch.to_int32()
    mask = oracle.partition(a, cfg.round_seed(0), cfg.S)
    p0, _ = synth.init_params(cfg.arch, cfg.init_seed)
    params = [p0.copy() for _ in range(cfg.S)]
    subs = cpu_sample(cfg)
    B, t = 2, oracle_step_all(cfg, a, mask, params, 2, 0, subs)
    if t < budget_s / 4:                                         # cheap network: a larger batch within the budget
        B = int(max(2, min(cfg.batch, 2 * budget_s / max(t, 1e-3))))
        t = oracle_step_all(cfg, a, mask, params, B, 1, subs)
    return {"value": len(subs) * B / t, "unit": "images/s", "cores": len(subs), "kind": "oracle",
            "sample": f"one local step of {len(subs)} of the S={cfg.S} sub-ResNets of the same network at batch {B} per sub-ResNet "
                      f"({t:.1f} s, one thread per sub-ResNet, {os.cpu_count()} host cores present)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg = workload_config(args)
    a = cfg.arch.to_int32()
    mask = oracle.partition(a, cfg.round_seed(0), cfg.S)
    p0, _ = synth.init_params(cfg.arch, cfg.init_seed)
    params = [p0.copy() for _ in range(cfg.S)]
    K, W = args.steps, args.warmup
    subs = cpu_sample(cfg)
    t2 = oracle_step_all(cfg, a, mask, params, 2, 0, subs)
    per_step = 150.0 / max(K + W, 1)                       # the whole run should end within a few minutes
    B = int(max(2, min(cfg.batch, 2 * per_step / max(t2, 1e-3))))
    if t2 > per_step and len(subs) > 1:                    # still too long at batch 2: fewer sub-ResNets per step
        subs = subs[:max(1, int(len(subs) * per_step / t2))]
    for i in range(W):
        oracle_step_all(cfg, a, mask, params, B, i, subs)
    t = 0.0
    for i in range(K):
        t += oracle_step_all(cfg, a, mask, params, B, W + i, subs)
    v = len(subs) * B * K / t
    sample = (f"each step = one local step of {len(subs)} of the S={cfg.S} sub-ResNets at batch {B} per sub-ResNet "
              f"(full workload: all {cfg.S} at batch {cfg.batch})")
    print(json.dumps({
        "impl": "reference", "metric": "sub-ResNet train images/s", "value": v, "unit": "images/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": W, "ms_per_step": 1e3 * t / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload][1] + "; CPU oracle on a bounded sample", "S": cfg.S, "batch_per_subnet": B},
        "cpu_baseline": {"value": v, "unit": "images/s", "cores": len(subs), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_reassembly(args):
    """Secondary measurement (not the headline line): the synchronisation step alone on the ResNet-101 parameter set
    (44.5 M fp32 parameters, bf16 shadow, momentum), S in {2, 4, 8}: `steps` calls of resist_aggregate and of
    resist_partition each, per-kernel CUDA-event times from the library, bandwidth against the measured HBM peak.
    The working copies hold the scattered global values (bandwidth does not depend on the values)."""
    import torch
    import paper_2107_00961_b200 as lib
    torch.cuda.set_device(0)
    cfg = synth.config(5)
    peaks = measured_peaks()
    ctx = lib.Context(cfg.arch.to_int32(), dtype=lib.BF16, momentum=0.9, seed=cfg.init_seed, device="cuda:0")
    K, W = args.steps, args.warmup
    out = {"metric": "reassembly and repartition bandwidth", "unit": "GB/s", "n_gpus": 1, "steps": K, "warmup": W, "dtype": "f32",
           "data": "synthetic", "config": {"workload": "configs[4]: reassembly / repartition stress on the ResNet-101 parameter set, S in {2,4,8}"},
           "peak_GBps": peaks["hbm_gbs"], "peak_source": peaks["source"], "by_S": {}}
    for S in (2, 4, 8):
        for i in range(W):
            ctx.partition(cfg.round_seed(100 * S + i), S)
            ctx.aggregate()
        torch.cuda.synchronize()
        ctx.set_profiling(True)
        ctx.get_profile()
        t0 = time.perf_counter()
        for i in range(K):
            ctx.partition(cfg.round_seed(1000 * S + i), S)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        for i in range(K):
            ctx.aggregate()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        prof = ctx.get_profile()
        ctx.set_profiling(False)
        rec = {"partition_call_us": (t1 - t0) / K * 1e6, "aggregate_call_us": (t2 - t1) / K * 1e6}
        for name in ("scatter", "aggregate"):
            v = prof[name]
            gbps = v["bytes"] / max(v["ms"], 1e-9) / 1e6
            rec[name] = {"us_per_call": v["ms"] / v["operations"] * 1e3, "MB_per_call": v["bytes"] / v["operations"] / 1e6, "GBps": gbps,
                         "frac_of_hbm_peak": gbps / peaks["hbm_gbs"]}
        out["by_S"][str(S)] = rec
    ctx.close()
    # the fused SGD-momentum update at a parameter count where bandwidth, not launch latency, is the time: a wide CIFAR
    # bottleneck net (the widths of configs[2] at reduced depth, 14 M parameters), S = 4, batch 2, grouped steps
    arch = synth.wide_cifar_arch(policy="stage_first_shared", depths=(2, 2, 2, 2))
    ctx = lib.Context(arch.to_int32(), dtype=lib.BF16, momentum=0.9, seed=1, device="cuda:0")
    S, B = 4, 2
    ctx.partition(11, S)
    xs = [torch.from_numpy(synth.round_to_bf16(synth.standard_normal(s, B * 32 * 32 * 3).astype(np.float32).reshape(B, 32, 32, 3))).cuda().to(torch.bfloat16)
          for s in range(S)]
    ys = [torch.zeros(B, dtype=torch.int32, device="cuda") for _ in range(S)]
    loss = torch.zeros(S, dtype=torch.float32, device="cuda")
    for _ in range(W):
        ctx.local_step_grouped(xs, ys, 0.1, loss)
    torch.cuda.synchronize()
    ctx.set_profiling(True)
    ctx.get_profile()
    for _ in range(min(K, 20)):
        ctx.local_step_grouped(xs, ys, 0.1, loss)
    v = ctx.get_profile()["sgd_momentum"]
    gbps = v["bytes"] / max(v["ms"], 1e-9) / 1e6
    out["sgd_momentum"] = {"params_per_subnet_held": v["bytes"] / v["operations"] / 22.0 / S, "us_per_call": v["ms"] / v["operations"] * 1e3,
                           "MB_per_call": v["bytes"] / v["operations"] / 1e6, "GBps": gbps, "frac_of_hbm_peak": gbps / peaks["hbm_gbs"]}
    print(json.dumps(out))


def run_micro(args):
    """tcgen05.mma rate on this device by MMA width, operand layout, number of issuing threads (see resist_micro_mma_rate)."""
    import torch
    import paper_2107_00961_b200 as lib
    torch.cuda.set_device(0)
    mhz = 1965.0
    rows = []
    names = {0: "K-major no swizzle", 1: "K-major 128B swizzle", 2: "K-major 128B swizzle, one 32-byte step", 3: "MN-major 128B swizzle"}
    for layout in (0, 1, 2, 3):
        for n in (16, 64, 128, 256):
            for issuers, alt in ((1, 0), (1, 1), (2, 0), (2, 1)):
                lib.micro_mma_rate(n, layout, 512, issuers, alt)
                c = min(lib.micro_mma_rate(n, layout, 4096, issuers, alt) for _ in range(3))
                rows.append({"layout": names[layout], "n": n, "issuers": issuers, "alternate_accumulators": alt, "cycles_per_mma": c,
                             "ideal_cycles": n / 2.0, "TFLOPs_per_gpu_at_max_clock": 2.0 * 128 * n * 16 / c * mhz * 1e6 * 148 / 1e12})
    print(json.dumps({"metric": "tcgen05.mma cycles per 128 x n x 16 MMA", "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wide", choices=["wide", "resnet110", "imagenet", "wide_localsgd", "reassembly", "micro"],
                    help="wide (default): the headline line; resnet110, imagenet: the other training configurations; wide_localsgd: the "
                         "local-SGD baseline on the wide network; reassembly: the synchronisation kernels alone")
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="leave the oracle's timing out of the line (quick kernel work)")
    ap.add_argument("--subnets", type=int, default=0, help="override S (smaller case of the same kernels for profiler captures)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch per sub-ResNet (likewise)")
    ap.add_argument("--profile-case", action="store_true", help="run W warm-up steps and one block of K steps only, print a short line (for ncu)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.workload == "micro":
        run_micro(args)
    elif args.workload == "reassembly":
        run_reassembly(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
