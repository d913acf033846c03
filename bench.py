#!/usr/bin/env python
"""Benchmark of the S-STE sparse linear hot path on B200.

One "step" = one pass of the whole path over one batch of the workload:
for every layer  project+compress -> sparse forward -> MVUE+compress ->
sparse grad_W -> dense grad_X  (beta is computed once, before timing: the paper
freezes it after the first iteration).  The default workload is the GPT-2-small
shaped MLP (two sparse linears, 8 x 1024 tokens, bf16).

Prints ONE JSON line.  `value` is dense-equivalent TFLOP/s (6*T*I*O per layer
per step) with all inputs resident in HBM; `e2e` is the same metric with the
inputs starting in pinned host memory and the gradients read back every step.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
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

METRIC = "S-STE linear fwd+bwd TFLOP/s (dense-equivalent)"
UNIT = "TFLOP/s"
KERNELS = ("project_compress", "linear_fwd", "mvue_sparsify", "linear_bwd_weight", "linear_bwd_input")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


def ncu_traffic(cfg_id: int, section: str = None):
    """DRAM bytes per launch (read + write) of each stage's kernel, from one ncu capture of this workload.

    The figures are measurements recorded in profiles/ncu_dram_traffic.json (with the command that produced
    them); a stage without a recorded capture reports null.
    """
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        return (rec.get(section, {}) if section else rec).get(f"config{cfg_id}", {})
    except (OSError, ValueError):
        return {}


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        super().__init__(daemon=True)
        self.gpu_index, self.samples, self.reasons, self.proc = gpu_index, [], set(), None
        self.max_mhz = None

    def run(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
            for line in self.proc.stdout:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    self.samples.append(float(parts[0]))
                    self.max_mhz = float(parts[1])
                except ValueError:
                    continue
                for name, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        self.reasons.add(name)
        except FileNotFoundError:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        load = sorted(self.samples)
        return {"sm_mhz": statistics.median(load) if load else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(load)}


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
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg_id = args.config
    cfg = workload_layers(cfg_id)
    tokens = min(cfg["layers"][0].T, args.ref_tokens)
    base, dt = time_oracle(cfg_id, tokens, args.steps, min(args.warmup, 1))
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
    return {"workload": f"BASELINE config {cfg_id}: " + ", ".join(f"{L.name} W[{L.O},{L.I}] x {L.T} tokens" for L in cfg["layers"]),
            "precision": "fp8 (e4m3 fwd / e5m2 bwd)" if cfg["fp8"] else "bf16",
            "tokens_per_gpu": cfg["layers"][0].T, "parallelism": f"dp{n_gpus} (token shards; grad_W all-reduced over NCCL when n_gpus > 1)",
            "l2": "flushed between timed steps (512 MiB write)", "launch": "n_gpus = 1: one CUDA-graph replay per step, grad_W on a side stream beside grad_X "
                      "(--no-overlap, --no-graph switch these off); n_gpus > 1: eager launches"}


# --------------------------------------------------------------------------------------------- GPU arm

def run_gpu(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2409_09099_b200 import binding as B, dp, synth
    from paper_2409_09099_b200.layer import SsteLinear

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg_id = args.config
    cfg = synth.CONFIGS[cfg_id]
    fp8 = cfg["fp8"]
    ctx = B.Context(local_rank)

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
        host.append(tuple(torch.from_numpy(a.view(np.int16)).pin_memory() for a in (W, X, dY)))
        flops_step += 6.0 * L.T * L.I * L.O
    torch.cuda.synchronize()

    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    overlap = not args.no_overlap and world == 1
    if overlap:
        ctx_side = B.Context(local_rank)
        side_stream = torch.cuda.Stream()

    def layer_step(li, step_idx, mark=lambda: None, serial=False):
        """The five calls of the path for one layer (+ the data-parallel exchange of its grad_W)."""
        lin, X, dY = layers[li]
        mark(); lin.prune()
        mark(); lin.forward(X)
        if overlap and not serial:
            mark(); lin.sparsify_grad(dY, step_idx, token_offset)
            mark(); mark()
            lin.grad_weight_and_input(dY, ctx_side, side_stream)
        else:
            mark(); lin.sparsify_grad(dY, step_idx, token_offset)
            mark(); lin.grad_weight()
            mark(); lin.grad_input(dY)
        mark()
        # data parallel: the per-rank partial grad_W is summed over ranks (the path's one exchange step)
        return dp.allreduce_grad_w([lin.dW])

    def step(step_idx, events=None):
        """All five calls for every layer; `events` (optional) collects per-kernel CUDA events."""
        def mark():
            if events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                events.append(e)
        handles = []
        for li in range(len(layers)):
            handles += layer_step(li, step_idx, mark, serial=events is not None)
        for h in handles:
            h.wait()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for w in range(max(args.warmup, 3)):
        step(w)
    barrier()

    # The timed step is one CUDA-graph replay of all launches of the step (no host work between kernels);
    # the MVUE step counter is frozen in the graph, which does not change the work done.
    graph = None
    if not args.no_graph and world == 1:      # collectives are launched eagerly
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(args.warmup)
        graph.replay()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    step_ms = []
    barrier()
    for s in range(args.steps):
        flush.zero_()                                   # evict L2 between timed steps
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        if graph is not None:
            graph.replay()
        else:
            step(args.warmup + s)
        e1.record(stream)
        torch.cuda.synchronize()
        step_ms.append(e0.elapsed_time(e1))
    barrier()
    # second timed pass, eager, with an event between kernels: the per-kernel breakdown and roofline
    per_kernel = {k: [] for k in KERNELS}
    n_before = B.launch_count()                         # the library counts its own kernel launches
    for s in range(args.steps):
        flush.zero_()
        ev = []
        step(args.warmup + s, ev)
        torch.cuda.synchronize()
        for li in range(len(layers)):
            base = li * 6
            for ki, k in enumerate(KERNELS):
                per_kernel[k].append((li, ev[base + ki].elapsed_time(ev[base + ki + 1])))
    launches_per_step = (B.launch_count() - n_before) // args.steps
    barrier()
    clocks = sampler.stop()
    gpu_launches = launches_per_step * args.steps       # libsste kernels executed in the K timed steps
    total_ms = sum(step_ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12

    # ---- end to end: inputs start in pinned host memory, gradients are read back ----
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
    e2e_steps = max(2, min(args.steps, 10))
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
    e2e_value = world * flops_step / (e2e_ms * 1e-3) / 1e12
    # ---- every stage on its own, hot: 10 calls back to back inside one CUDA graph (no launch or event gaps,
    # operands L2-resident where they fit) -- the kernel-level companion of the per-stage times above
    hot_us = {}
    if world == 1:
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
    status = ctx.poll_device_status()

    if rank == 0:
        peaks = measured_peaks()
        # Share of each stage of the path in the eager timed pass, and its roofline.  A stage is one C-ABI
        # call of the path (for FP8 together with the amax / scale / quantise helpers that precede it).
        tot = {k: sum(ms for _, ms in v) for k, v in per_kernel.items()}
        Ls = cfg["layers"]
        traffic = ncu_traffic(cfg_id)
        alu_pct = ncu_traffic(cfg_id, "alu_pipe_pct")
        rooflines = {}
        for k in KERNELS:
            avg_ms = tot[k] / len(per_kernel[k])
            if k in ("linear_fwd", "linear_bwd_weight", "linear_bwd_input"):
                fl = sum(2.0 * L.T * L.I * L.O for L in Ls) / len(Ls)       # dense-equivalent flops per launch (mean)
                sparse = k != "linear_bwd_input"
                # peak of the kernel's own dtype: measured bf16 dense x nominal ratios (2:4 sparse x2, fp8 x2)
                peak = peaks["bf16_tflops"] * (2.0 if sparse else 1.0) * (2.0 if fp8 else 1.0)
                ach = fl / (avg_ms * 1e-3) / 1e12
                # compulsory HBM bytes per launch (operands once in, result once out): the floor of a thin product
                eb = 1 if fp8 else 2
                byt = sum((L.T * L.I * eb + L.O * L.I * (eb * (0.5 if sparse else 1.0) + (0.125 if sparse else 0.0))
                           + L.T * L.O * 2) if k == "linear_fwd" else
                          (L.O * L.T * (eb * 0.5 + 0.125) + L.T * L.I * eb + L.O * L.I * 2) if k == "linear_bwd_weight" else
                          (L.T * L.O * eb + L.O * L.I * eb + L.T * L.I * 2) for L in Ls) / len(Ls)
                rooflines[k] = {"kernel": k, "bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                                "frac": ach / peak, "traffic": traffic.get(k),
                                "us_per_launch": avg_ms * 1e3, "us_per_launch_hot": hot_us.get(k),
                                "frac_hot": (fl / (hot_us[k] * 1e-6) / 1e12 / peak) if k in hot_us else None,
                                "tensor_floor_us": fl / (peak * 1e12) * 1e6,
                                "hbm_floor_us": byt / (peaks["hbm_gbs"] * 1e9) * 1e6,
                                "peak_source": f"{peaks['source']} cuBLAS bf16 dense burst"
                                               + (" x2 (2:4 sparse, nominal ratio)" if sparse else "")
                                               + (" x2 (fp8, nominal ratio)" if fp8 else "")}
            else:
                # algorithmic bytes per element: read bf16 + compressed values + metadata (+ dense copy)
                if k == "project_compress":
                    per_elt, elts = (3.625 if fp8 else 5.125), sum(L.O * L.I for L in Ls) / len(Ls)
                else:
                    per_elt, elts = (3.625 if fp8 else 3.125), sum(L.T * L.O for L in Ls) / len(Ls)
                ach = per_elt * elts / (avg_ms * 1e-3) / 1e9
                rooflines[k] = {"kernel": k, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": ach / peaks["hbm_gbs"], "traffic": traffic.get(k),
                                "us_per_launch": avg_ms * 1e3, "us_per_launch_hot": hot_us.get(k),
                                "frac_hot": (per_elt * elts / (hot_us[k] * 1e-6) / 1e9 / peaks["hbm_gbs"])
                                if k in hot_us else None,
                                "hbm_floor_us": per_elt * elts / (peaks["hbm_gbs"] * 1e9) * 1e6,
                                # ncu: share of the half-rate integer/compare pipe while the kernel runs -- these
                                # kernels are bound by it, not by HBM
                                "alu_pipe_pct_ncu": alu_pct.get(k),
                                "peak_source": f"{peaks['source']} copy bandwidth"}
        dom = max(tot, key=tot.get)
        roofline = rooflines[dom]
        breakdown = {k: {"ms_per_step": tot[k] / args.steps, "share": tot[k] / sum(tot.values()),
                         "roofline_frac": rooflines[k]["frac"], "bound": rooflines[k]["bound"]} for k in KERNELS}
        cpu_base = None
        if world == 1 or rank == 0:
            cpu_base, _ = time_oracle(cfg_id, min(cfg["layers"][0].T, args.ref_tokens), 5, 1)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "ms_per_step_median": statistics.median(step_ms), "ms_per_step_min": min(step_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8" if fp8 else "bf16", "data": "synthetic",
            "config": workload_config(cfg_id, cfg, world),
            # whole step (sparse and dense products, elementwise kernels) against the nominal 2:4 sparse peak
            "pct_of_sparse_peak_nominal": 100.0 * value / world / (9000.0 if fp8 else 4500.0),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "overlap": "copies in, compute and copies out on three streams, ordered by events"},
            "gpu_launches": gpu_launches,
            "roofline": roofline,
            "rooflines": rooflines,
            "kernels": breakdown,
            "cpu_baseline": cpu_base,
            "device_status": status,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="BASELINE config id (2 = GPT-2-small MLP, the default workload)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="run grad_W and grad_X back to back instead of grad_W on a side stream beside grad_X")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps eagerly instead of replaying a CUDA graph")
    ap.add_argument("--ref-tokens", type=int, default=8192, help="tokens per layer in the CPU-oracle sample")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
