#!/usr/bin/env python
"""Benchmark of the S-STE sparse linear hot path on B200.

One "step" = one pass of the whole path over one batch of the workload:
for every layer  project+compress -> sparse forward -> MVUE+compress ->
sparse grad_W -> dense grad_X  (beta is computed once, before timing: the paper
freezes it after the first iteration).  The default workload is the largest
single-GPU configuration, the FP8 whole-process variant on a 7B-shaped FFN
(config 5); the same run also measures the two bf16 workloads (configs 2 and 3)
and reports them under `per_config`.

Prints ONE JSON line.  `value` is dense-equivalent TFLOP/s (6*T*I*O per layer
per step) with all inputs resident in HBM; `e2e` is the same metric with the
inputs starting in pinned host memory and the gradients read back every step.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
`--gpus N` without a torchrun environment starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "S-STE linear fwd+bwd TFLOP/s (dense-equivalent)"
UNIT = "TFLOP/s"
# stages of the path and the C-ABI calls (labels of SsteLinear.mark) that belong to each
STAGES = {
    "project_compress": ("project_amax", "project_compress"),
    "linear_fwd": ("amax_x", "quantize_x", "linear_fwd"),
    "mvue_sparsify": ("amax_g", "mvue_sparsify"),
    "linear_bwd_weight": ("linear_bwd_weight",),
    "linear_bwd_input": ("linear_bwd_input",),
}
NOMINAL = dict(hbm_gbs=8000.0, bf16_dense=2250.0)   # the figures the task names: ~8 TB/s, 2.25 PFLOP/s dense bf16


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


def ncu_record(cfg_id: int, section: str = "dram_bytes"):
    """Per-stage figures from ncu captures of this workload, recorded in profiles/ncu_dram_traffic.json (with the
    commands that produced them); a stage without a recorded capture reports null."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        return rec.get(section, {}).get(f"config{cfg_id}", {})
    except (OSError, ValueError):
        return {}


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi for the whole run; windows are cut by host time."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_index: int):
        super().__init__(daemon=True)
        self.gpu_index, self.samples, self.proc, self.max_mhz = gpu_index, [], None, None

    def run(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    mhz, self.max_mhz, watts = float(parts[0]), float(parts[1]), float(parts[2])
                except ValueError:
                    continue
                reasons = [n for n, v in zip(self.NAMES, parts[3:7]) if v.lower().startswith("active")]
                self.samples.append((time.time(), mhz, watts, reasons))
        except FileNotFoundError:
            pass

    def window(self, t0: float, t1: float):
        """Clock record of the host-time window [t0, t1]."""
        w = [s for s in list(self.samples) if t0 <= s[0] <= t1]
        reasons = sorted({r for s in w for r in s[3]})
        return {"sm_mhz": statistics.median(s[1] for s in w) if w else None, "sm_max_mhz": self.max_mhz,
                "power_w_max": max((s[2] for s in w), default=None), "reasons": reasons, "samples": len(w)}

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)


def workload_layers(cfg_id: int):
    from paper_2409_09099_b200 import synth
    return synth.CONFIGS[cfg_id]


# --------------------------------------------------------------------------------------------- CPU oracle arm

def oracle_step(tensors, seed, step, fp8=False):
    """One pass of the path on the CPU oracle for a list of (W, X, dY, beta32) samples."""
    from oracle import sste_oracle as orc
    for li, (W, X, dY, beta32) in enumerate(tensors):
        if fp8:   # whole-process FP8: per-tensor scales, E4M3 forward operands, E5M2 gradient
            _, _, wt = orc.project_compress(W, beta32)
            sw, sx, sg = (orc.fp8_scale(orc.amax(wt), orc.E4M3), orc.fp8_scale(orc.amax(X), orc.E4M3),
                          orc.fp8_scale(orc.amax(dY), orc.E5M2))
            vals, meta, dense = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=sw)
            Xq = orc.quantize(X, sx, orc.E4M3)
            orc.linear_fwd(Xq, orc.E4M3, vals, meta, orc.E4M3, 1.0 / (float(sx) * float(sw)))
            gv, gm, dq, _ = orc.mvue(dY, seed, li, step, odt=orc.E5M2, gscale=sg, want_dense_q=True)
            orc.linear_bwd_weight(gv, gm, orc.E5M2, Xq, orc.E4M3, 1.0 / (float(sg) * float(sx)))
            orc.linear_bwd_input(dq, orc.E5M2, dense, orc.E4M3, 1.0 / (float(sg) * float(sw)))
            continue
        vals, meta, dense = orc.project_compress(W, beta32)
        orc.linear_fwd(X, orc.BF16, vals, meta, orc.BF16)
        gv, gm, _, _ = orc.mvue(dY, seed, li, step)
        orc.linear_bwd_weight(gv, gm, orc.BF16, X, orc.BF16)
        orc.linear_bwd_input(dY, orc.BF16, dense, orc.BF16)


def oracle_tokens(cfg_id: int, budget_flops: float) -> int:
    """Tokens per layer of the bounded CPU sample: the full batch if it fits the budget, else a multiple of 128."""
    cfg = workload_layers(cfg_id)
    per_token = sum(6.0 * L.I * L.O for L in cfg["layers"])
    T = cfg["layers"][0].T
    return int(max(128, min(T, int(budget_flops / per_token) // 128 * 128)))


def oracle_sample(cfg_id: int, tokens: int):
    import numpy as np
    from oracle import sste_oracle as orc
    from paper_2409_09099_b200 import synth
    cfg = synth.CONFIGS[cfg_id]
    tensors, flops = [], 0.0
    for li, L in enumerate(cfg["layers"]):
        W, X, dY = synth.layer_tensors(cfg_id, li, T=tokens)
        tensors.append((W, X, dY, np.float32(orc.beta(W)[0])))
        flops += 6.0 * tokens * L.I * L.O
    return cfg, tensors, flops


def time_oracle(cfg_id: int, tokens: int, steps: int, warmup: int):
    cfg, tensors, flops = oracle_sample(cfg_id, tokens)
    for w in range(warmup):
        oracle_step(tensors, cfg["seed"], w, cfg["fp8"])
    t0 = time.perf_counter()
    for s in range(steps):
        oracle_step(tensors, cfg["seed"], s, cfg["fp8"])
    dt = (time.perf_counter() - t0) / max(steps, 1)
    cores = len(os.sched_getaffinity(0))
    return dict(value=flops / dt / 1e12, unit=UNIT, cores=cores, kind="oracle",
                sample=f"config {cfg_id} with {tokens} of {cfg['layers'][0].T} tokens per layer, "
                       f"{steps} step(s), {dt:.2f} s per step"), dt


def run_reference(args):
    """The CPU oracle as it stands on the host cores: rank 0 alone works and prints."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg_id = args.config
    cfg = workload_layers(cfg_id)
    tokens = args.ref_tokens or oracle_tokens(cfg_id, 0.4e12)
    base, dt = time_oracle(cfg_id, min(cfg["layers"][0].T, tokens), args.steps, min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg_id, cfg, 1),
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg_id, cfg, n_gpus):
    return {"workload": f"config {cfg_id}: " + ", ".join(f"{L.name} W[{L.O},{L.I}] x {L.T} tokens" for L in cfg["layers"]),
            "precision": "fp8 (e4m3 fwd / e5m2 bwd)" if cfg["fp8"] else "bf16",
            "tokens_per_gpu": cfg["layers"][0].T, "parallelism": f"dp{n_gpus} (token shards; grad_W all-reduced over NCCL when n_gpus > 1)",
            "l2": "flushed between timed steps (512 MiB write)", "launch": "n_gpus = 1: one CUDA-graph replay per step, grad_W on a side stream beside grad_X "
                      "(--no-overlap, --no-graph switch these off); n_gpus > 1: eager launches"}


# --------------------------------------------------------------------------------------------- GPU arm

def stage_rooflines(cfg, per_call_us, hot_us, peaks, cfg_id):
    """Roofline of every stage of the path from the event-timed eager pass (`per_call_us`: label -> mean
    microseconds per call) and the back-to-back graph timing (`hot_us`: stage -> microseconds)."""
    fp8, Ls = cfg["fp8"], cfg["layers"]
    traffic, alu_pct = ncu_record(cfg_id), ncu_record(cfg_id, "alu_pipe_pct")
    out = {}
    for stage, labels in STAGES.items():
        main = labels[-1]
        us = per_call_us.get(main)
        helpers = {l: per_call_us[l] for l in labels[:-1] if l in per_call_us}
        if us is None:
            continue
        if stage.startswith("linear_"):
            fl = sum(2.0 * L.T * L.I * L.O for L in Ls) / len(Ls)       # dense-equivalent flops per launch (mean)
            sparse = stage != "linear_bwd_input"
            # peak of the kernel's own dtype: measured bf16 dense x nominal ratios (2:4 sparse x2, fp8 x2)
            mult = (2.0 if sparse else 1.0) * (2.0 if fp8 else 1.0)
            peak, nominal = peaks["bf16_tflops"] * mult, NOMINAL["bf16_dense"] * mult
            ach = fl / (us * 1e-6) / 1e12
            eb = 1 if fp8 else 2
            # compulsory HBM bytes per launch (operands once in, result once out): the floor of a thin product
            byt = sum((L.T * L.I * eb + L.O * L.I * (eb * 0.5 + 0.125) + L.T * L.O * 2) if stage == "linear_fwd" else
                      (L.O * L.T * (eb * 0.5 + 0.125) + L.T * L.I * eb + L.O * L.I * 2) if stage == "linear_bwd_weight" else
                      (L.T * L.O * eb + L.O * L.I * eb + L.T * L.I * 2) for L in Ls) / len(Ls)
            out[stage] = {"kernel": stage, "bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                          "frac": ach / peak, "frac_nominal": ach / nominal, "peak_nominal": nominal,
                          "traffic": traffic.get(stage), "us_per_launch": us, "helpers_us": helpers,
                          "us_per_launch_hot": hot_us.get(stage),
                          "frac_hot": (fl / (hot_us[stage] * 1e-6) / 1e12 / peak) if stage in hot_us else None,
                          "tensor_floor_us": fl / (peak * 1e12) * 1e6,
                          "hbm_floor_us": byt / (peaks["hbm_gbs"] * 1e9) * 1e6,
                          "peak_source": f"{peaks['source']} cuBLAS bf16 dense burst"
                                         + (" x2 (2:4 sparse, nominal ratio)" if sparse else "")
                                         + (" x2 (fp8, nominal ratio)" if fp8 else "")}
        else:
            # algorithmic bytes per element: read bf16 + compressed values + metadata + the dense copy (w~ for grad_X;
            # FP8: the E5M2 copy of dY)
            if stage == "project_compress":
                per_elt, elts = (3.625 if fp8 else 5.125), sum(L.O * L.I for L in Ls) / len(Ls)
            else:
                per_elt, elts = (3.625 if fp8 else 3.125), sum(L.T * L.O for L in Ls) / len(Ls)
            ach = per_elt * elts / (us * 1e-6) / 1e9
            out[stage] = {"kernel": stage, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL["hbm_gbs"],
                          "peak_nominal": NOMINAL["hbm_gbs"], "traffic": traffic.get(stage),
                          "us_per_launch": us, "helpers_us": helpers, "us_per_launch_hot": hot_us.get(stage),
                          "frac_hot": (per_elt * elts / (hot_us[stage] * 1e-6) / 1e9 / peaks["hbm_gbs"])
                          if stage in hot_us else None,
                          "bytes_per_element": per_elt,
                          "hbm_floor_us": per_elt * elts / (peaks["hbm_gbs"] * 1e9) * 1e6,
                          # ncu: share of the half-rate integer/compare pipe while the kernel runs
                          "alu_pipe_pct_ncu": alu_pct.get(stage),
                          "peak_source": f"{peaks['source']} copy bandwidth"}
    return out


def measure_config(cfg_id, args, env, full):
    """All measurements of one workload.  `full`: also end to end, per-stage hot timings and the CPU baseline."""
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2409_09099_b200 import binding as B, dp, synth
    from paper_2409_09099_b200.layer import SsteLinear

    rank, world, local_rank, sampler = env["rank"], env["world"], env["local_rank"], env["sampler"]
    dev = f"cuda:{local_rank}"
    cfg = synth.CONFIGS[cfg_id]
    fp8 = cfg["fp8"]
    ctx = B.Context(local_rank)
    steps = args.steps

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    # weak scaling: every rank holds the full weights and its own batch of tokens (seeded per rank); the
    # global batch is world x T tokens and a rank's MVUE counter starts at its first token
    token_offset = rank * cfg["layers"][0].T
    layers, host = [], []
    flops_step = 0.0
    for li, L in enumerate(cfg["layers"]):
        W, X, dY = synth.layer_tensors(cfg_id, li)
        if rank > 0:
            X = synth.gaussian_bf16(cfg["seed"] * 1000 + 10 * li + 1 + 100 * rank, X.shape, L.sigma_x)
            dY = synth.gaussian_bf16(cfg["seed"] * 1000 + 10 * li + 2 + 100 * rank, dY.shape, L.sigma_g)
        lin = SsteLinear(ctx, to_dev(W), L.T, tensor_id=li, seed=cfg["seed"], fp8=fp8)
        lin.init_beta()
        layers.append((lin, to_dev(X), to_dev(dY)))
        if full:
            host.append(tuple(torch.from_numpy(a.view(np.int16)).pin_memory() for a in (W, X, dY)))
        flops_step += 6.0 * L.T * L.I * L.O
    torch.cuda.synchronize()

    flush = env["flush"]
    stream = torch.cuda.current_stream()
    overlap = not args.no_overlap and world == 1
    if overlap:
        ctx_side = B.Context(local_rank)
        side_stream = torch.cuda.Stream()

    def layer_step(li, step_idx, serial=False):
        """The calls of the path for one layer (+ the data-parallel exchange of its grad_W)."""
        lin, X, dY = layers[li]
        lin.prune()
        lin.forward(X)
        lin.sparsify_grad(dY, step_idx, token_offset)
        if overlap and not serial:
            lin.grad_weight_and_input(dY, ctx_side, side_stream)
        else:
            lin.grad_weight()
            lin.grad_input(dY)
        # data parallel: the per-rank partial grad_W is summed over ranks (the path's one exchange step)
        return dp.allreduce_grad_w([lin.dW])

    def step(step_idx, serial=False):
        handles = []
        for li in range(len(layers)):
            handles += layer_step(li, step_idx, serial)
        for h in handles:
            h.wait()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def check_status(what):
        st = ctx.poll_device_status()
        if st != 0:
            raise RuntimeError(f"libsste recorded device status {st} during {what}: the timing is void")

    warm = max(args.warmup, 3)
    for w in range(warm):
        step(w)
    barrier()
    check_status("warm-up")

    # The timed step is one CUDA-graph replay of all launches of the step (no host work between kernels);
    # the MVUE step counter is frozen in the graph, which does not change the work done.
    graph = None
    if not args.no_graph and world == 1:      # collectives are launched eagerly
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(warm)
        graph.replay()
        torch.cuda.synchronize()

    # ---- timed region: EXACTLY `steps` steps per repeat, L2 flushed before every step, CUDA events on the
    # launching stream; repeated until at least one second of steps has been timed
    t_host0 = time.time()
    n_before = B.launch_count()
    repeat_ms, all_ms = [], []
    while True:
        barrier()
        ms = []
        for s in range(steps):
            flush.zero_()                                   # evict L2 between timed steps
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            if graph is not None:
                graph.replay()
            else:
                step(warm + s)
            e1.record(stream)
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        barrier()
        repeat_ms.append(sum(ms))
        all_ms += ms
        if sum(repeat_ms) >= args.min_timed_ms or len(repeat_ms) >= 400:
            break
    t_host1 = time.time()
    eager_launches = B.launch_count() - n_before           # 0 under graph replay: the graph holds the launches
    check_status("the timed region")
    repeats = len(repeat_ms)
    per_rep = repeat_ms
    if world > 1:       # max over ranks of every repeat
        t = torch.tensor(per_rep, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        per_rep = t.tolist()
    ms_per_step = sum(per_rep) / (repeats * steps)
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12
    clocks = sampler.window(t_host0, t_host1)

    if args.timed_only:        # a profiler run: the warm-up and the timed steps only
        ctx.close()
        return {"value": value, "unit": UNIT, "ms_per_step": ms_per_step, "repeats": repeats, "timed_only": True,
                "dtype": "fp8" if fp8 else "bf16", "config": workload_config(cfg_id, cfg, world), "clocks": clocks}

    # ---- sustained: graph replays back to back for two seconds, no flush, no host gaps: what a training loop sees
    sustained = None
    if graph is not None:
        n_rep = max(5, int(args.sustained_ms / ms_per_step))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ts0 = time.time()
        e0.record(stream)
        for _ in range(n_rep):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        ts1 = time.time()
        sus_ms = e0.elapsed_time(e1) / n_rep
        sclk = sampler.window(ts0 + 0.2 * (ts1 - ts0), ts1)     # skip the ramp
        sustained = {"ms_per_step": sus_ms, "value": flops_step / (sus_ms * 1e-3) / 1e12, "unit": UNIT, "steps": n_rep,
                     "seconds": ts1 - ts0, "clocks": sclk,
                     "mclk_per_step": sus_ms * sclk["sm_mhz"] * 1e-3 if sclk["sm_mhz"] else None,
                     "note": "no L2 flush, no host gaps; mclk_per_step = ms x median SM MHz (clock-normalised time)"}
        check_status("the sustained loop")

    # ---- second pass, eager, with an event before every C-ABI call: the per-call breakdown and rooflines
    marks = []

    def mark(label):
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        marks.append((label, e))

    for lin, _, _ in layers:
        lin.mark = mark
    n_before = B.launch_count()
    per_call = {}
    k_steps = min(steps, 10)
    for s in range(k_steps):
        flush.zero_()
        marks.clear()
        for li in range(len(layers)):
            for h in layer_step(li, warm + s, serial=True):
                h.wait()
        mark("end")
        torch.cuda.synchronize()
        for (label, e), (_, e_next) in zip(marks[:-1], marks[1:]):
            per_call.setdefault(label, []).append(e.elapsed_time(e_next) * 1e3)
    launches_per_step = (B.launch_count() - n_before) // k_steps
    for lin, _, _ in layers:
        lin.mark = None
    check_status("the per-call pass")
    per_call_us = {k: sum(v) / len(v) for k, v in per_call.items()}            # mean over layers and steps
    per_call_step_us = {k: sum(v) / k_steps for k, v in per_call.items()}      # per step, all layers together
    gpu_launches = launches_per_step * steps * repeats       # libsste kernels executed in the timed region

    # ---- every stage on its own, hot: 10 calls back to back inside one CUDA graph
    hot_us = {}
    if world == 1 and full:
        calls = {
            "project_compress": lambda lin, X, dY: lin.prune(),
            "linear_fwd": lambda lin, X, dY: lin.forward(X),
            "mvue_sparsify": lambda lin, X, dY: lin.sparsify_grad(dY, 0, token_offset),
            "linear_bwd_weight": lambda lin, X, dY: lin.grad_weight(),
            "linear_bwd_input": lambda lin, X, dY: lin.grad_input(dY),
        }
        reps = 10
        for k, fn in calls.items():
            per_layer = []
            for lin, X, dY in layers:
                fn(lin, X, dY)
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for _ in range(reps):
                        fn(lin, X, dY)
                g.replay()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                g.replay()
                e1.record(stream)
                torch.cuda.synchronize()
                per_layer.append(e0.elapsed_time(e1) / reps * 1e3)
                del g
            hot_us[k] = sum(per_layer) / len(per_layer)
        check_status("the per-stage hot timing")

    # ---- end to end: inputs start in pinned host memory, gradients are read back ----
    e2e = None
    if full:
        h2d = sum(sum(t.numel() * 2 for t in h) for h in host)
        outs = [(torch.empty(l.dW.shape, dtype=torch.int16).pin_memory(), torch.empty(l.dX.shape, dtype=torch.int16).pin_memory())
                for l, _, _ in layers]
        d2h = sum(a.numel() * 2 + b.numel() * 2 for a, b in outs)
        # Three streams: host->device copies, the path, device->host copies.  Per layer, a step's inputs are
        # copied while the previous layer computes and the previous results are read back (PCIe is full duplex);
        # events order the reuse of every buffer, so each step still moves and computes everything.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        nl = len(layers)
        ev_in = [torch.cuda.Event() for _ in range(nl)]      # inputs of layer l are on the device
        ev_comp = [torch.cuda.Event() for _ in range(nl)]    # layer l has consumed its inputs and produced its outputs
        ev_out = [torch.cuda.Event() for _ in range(nl)]     # outputs of layer l are on the host
        for e in ev_comp + ev_out:
            e.record(stream)

        def e2e_step(step_idx):
            for li, ((lin, X, dY), (hW, hX, hdY)) in enumerate(zip(layers, host)):
                s_in.wait_event(ev_comp[li])
                with torch.cuda.stream(s_in):
                    lin.W.view(torch.int16).copy_(hW, non_blocking=True)
                    X.view(torch.int16).copy_(hX, non_blocking=True)
                    dY.view(torch.int16).copy_(hdY, non_blocking=True)
                    ev_in[li].record(s_in)
            for li, ((lin, _, _), (oW, oX)) in enumerate(zip(layers, outs)):
                stream.wait_event(ev_in[li])
                stream.wait_event(ev_out[li])
                for h in layer_step(li, step_idx):
                    h.wait()
                ev_comp[li].record(stream)
                s_out.wait_event(ev_comp[li])
                with torch.cuda.stream(s_out):
                    oW.copy_(lin.dW.view(torch.int16), non_blocking=True)
                    oX.copy_(lin.dX.view(torch.int16), non_blocking=True)
                    ev_out[li].record(s_out)

        def e2e_drain():
            for e in ev_out:
                stream.wait_event(e)

        e2e_step(0)
        e2e_drain()
        barrier()
        e2e_steps = max(2, min(steps, 10, int(1500.0 / max(h2d / 20e6, 1.0)) or 2))   # about 1.5 s of PCIe traffic
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for s in range(e2e_steps):
            e2e_step(s)
        e2e_drain()
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        if world > 1:
            t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        check_status("the end-to-end loop")
        e2e = {"value": world * flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "overlap": "copies in, compute and copies out on three streams, ordered by events"}
        del outs, host

    peaks = measured_peaks()
    rooflines = stage_rooflines(cfg, per_call_us, hot_us, peaks, cfg_id)
    stage_us = {st: sum(per_call_step_us.get(l, 0.0) for l in labels) for st, labels in STAGES.items()}
    total_us = sum(stage_us.values()) or 1.0
    # the dominant KERNEL: the stage whose main kernel (helpers apart) takes the most time per step
    dom = max(STAGES, key=lambda st: per_call_step_us.get(STAGES[st][-1], 0.0))
    breakdown = {st: {"ms_per_step": stage_us[st] * 1e-3, "share": stage_us[st] / total_us,
                      "roofline_frac": rooflines[st]["frac"], "bound": rooflines[st]["bound"]} for st in STAGES}
    rep_ms = [r / steps for r in per_rep]
    result = {
        "value": value, "unit": UNIT, "ms_per_step": ms_per_step, "repeats": repeats,
        "ms_per_step_median": statistics.median(rep_ms), "ms_per_step_min": min(rep_ms),
        "ms_per_step_single_min": min(all_ms), "timed_ms": sum(per_rep),
        "dtype": "fp8" if fp8 else "bf16",
        "config": workload_config(cfg_id, cfg, world),
        # whole step (sparse and dense products, elementwise kernels) against the nominal 2:4 sparse peak
        "pct_of_sparse_peak_nominal": 100.0 * value / world / (9000.0 if fp8 else 4500.0),
        "clocks": clocks, "sustained": sustained, "e2e": e2e, "gpu_launches": gpu_launches,
        "launches_per_step": launches_per_step, "eager_launches_in_timed_region": eager_launches,
        "roofline": rooflines[dom], "rooflines": rooflines, "kernels": breakdown,
        "calls_us": per_call_us,
    }
    for lin, _, _ in layers:
        del lin
    layers.clear()
    ctx.close()
    if overlap:
        ctx_side.close()
    torch.cuda.empty_cache()
    return result


def run_gpu(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        # the communicator log (rings / trees, NVLS or not) goes to stderr; stdout carries the one JSON line
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT,GRAPH")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=torch.device(dev))
    sampler = ClockSampler(local_rank)
    sampler.start()
    env = dict(rank=rank, world=world, local_rank=local_rank, sampler=sampler,
               flush=torch.empty(512 << 20, dtype=torch.uint8, device=dev))
    time.sleep(0.3)

    main = measure_config(args.config, args, env, full=True)
    per_config = {}
    if world == 1 and not args.no_per_config and not args.timed_only:
        for other in (2, 3):
            if other != args.config:
                r = measure_config(other, args, env, full=False)
                per_config[str(other)] = {k: r[k] for k in ("value", "unit", "ms_per_step", "ms_per_step_median",
                                                            "ms_per_step_min", "repeats", "dtype", "config",
                                                            "pct_of_sparse_peak_nominal", "clocks", "sustained",
                                                            "rooflines", "kernels", "launches_per_step")}
    sampler.stop()

    if rank == 0 and args.timed_only:
        print(json.dumps(main), flush=True)
    elif rank == 0:
        cpu_tokens = args.ref_tokens or oracle_tokens(args.config, 1.0e12)
        cpu_base, _ = time_oracle(args.config, cpu_tokens, 3, 1)
        line = {
            "metric": METRIC, "value": main["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": main["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "data": "synthetic",
        }
        line.update({k: v for k, v in main.items() if k not in line})
        line["per_config"] = per_config
        line["cpu_baseline"] = cpu_base
        line["device_status"] = 0
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_model(args):
    """--config 4: training steps of the 12-layer GPT-2-124M-shaped decoder with every linear through libsste."""
    import torch

    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.model import SsteGpt2, synthetic_batch
    torch.cuda.set_device(0)
    sampler = ClockSampler(0)
    sampler.start()
    ctx = B.Context(0)
    model = SsteGpt2(ctx)
    tokens, targets = synthetic_batch(model, 4)
    for _ in range(max(args.warmup, 3)):
        model.train_step(tokens, targets)
    torch.cuda.synchronize()
    n0, t0 = B.launch_count(), time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        loss, _ = model.train_step(tokens, targets)
    e1.record()
    torch.cuda.synchronize()
    t1, launches = time.time(), B.launch_count() - n0
    ms = e0.elapsed_time(e1) / args.steps
    inside, total = 0.0, 0.0
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        _, t_in = model.train_step(tokens, targets, time_libsste=True)
        b.record()
        torch.cuda.synchronize()
        inside, total = inside + t_in, total + a.elapsed_time(b) * 1e-3
    status = ctx.poll_device_status()
    sampler.stop()
    line = {"metric": METRIC, "value": model.flops_per_step() / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "config 4: 12-layer GPT-2-124M-shaped decoder, 8 x 1024 uniform token ids, all 48 "
                                   "linears through libsste; attention, layer norms, embeddings, loss and AdamW in torch",
                       "note": "value counts the S-STE linears' 6*T*I*O flops over the WHOLE training step"},
            "libsste_fraction_of_step": inside / total, "loss": float(loss), "gpu_launches": int(launches),
            "clocks": sampler.window(t0, t1), "device_status": status}
    print(json.dumps(line), flush=True)


def spawn_ranks(args):
    """`--gpus N` outside a torchrun environment: start the N ranks (one per GPU) and let rank 0 print."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5,
                    help="benchmark config id (5 = FP8 7B-shaped FFN, the largest single-GPU workload; 2, 3 bf16)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="run grad_W and grad_X back to back instead of grad_W on a side stream beside grad_X")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-per-config", action="store_true", help="measure only --config, not the other bf16 workloads")
    ap.add_argument("--timed-only", action="store_true",
                    help="stop after the timed steps (for profiler runs: few launches, no end-to-end / CPU legs)")
    ap.add_argument("--min-timed-ms", type=float, default=1000.0, help="repeat the K timed steps until this much is timed")
    ap.add_argument("--sustained-ms", type=float, default=2000.0, help="length of the back-to-back sustained loop")
    ap.add_argument("--ref-tokens", type=int, default=0, help="tokens per layer in the CPU-oracle sample (0 = sized to a budget)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.config == 4:
        run_model(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
