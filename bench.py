#!/usr/bin/env python
"""Benchmark of the SignMuon optimizer step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

A "step" is one full optimizer step (momentum, Newton-Schulz, sign+pack, vote, update) over one
set of synthetic per-worker gradients.  Default workload: the ResNet-50-shaped parameter set
(54 matrices, fp32, M = 4 workers, K = 5 Newton-Schulz steps).  Prints ONE JSON line.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent
replica of the same step ("replicas only": the worker axis is simulated on each GPU, there is no
exchange step to shard); the value is the sum over ranks, timed as the max over ranks.

--impl reference times the float64 CPU oracle on a bounded sample of the same workload.
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

METRIC = "signmuon_optimizer_steps_per_sec"
UNIT = "steps/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def oracle_sample_plan(wl, budget_flops=1.2e11):
    """Chooses a prefix-by-cost sample of the workload's parameters whose literal float64
    Newton-Schulz work stays near `budget_flops`, and returns (indices, sample_cost, total_cost)."""
    def cost(p):
        base = 10.0 * p.numel * wl.num_workers
        if p.kind != "matrix":
            return base
        c = 4.0 * p.cols * p.cols * p.rows * wl.ns_steps * (wl.num_workers + (1 if wl.local_polar else 0))
        return base + c
    costs = [cost(p) for p in wl.params]
    total = sum(costs)
    order = sorted(range(len(costs)), key=lambda i: costs[i])
    chosen, acc = [], 0.0
    # spread over the size range: walk from cheap to expensive, taking every other parameter
    for i in order[::2]:
        if acc + costs[i] > budget_flops and chosen:
            continue
        chosen.append(i)
        acc += costs[i]
    return sorted(chosen), acc, total


def time_oracle(wl, steps, warmup, budget_flops):
    import numpy as np
    import torch
    import oracle as O
    from threadpoolctl import threadpool_info
    from paper_2605_16311_b200 import workloads as wlmod

    idx, c_sample, c_total = oracle_sample_plan(wl, budget_flops)
    sub = wlmod.Workload(wl.name + "_oracle_sample", [wl.params[i] for i in idx], wl.num_workers, wl.momentum, wl.lr,
                         wl.ns_steps, wl.local_polar, wl.steps, wl.signal_std, wl.noise_std, wl.noise,
                         wl.weight_std, wl.config_id)
    specs = [O.ParamSpec(p.rows, p.cols, p.kind, p.dtype) for p in sub.params]
    cfg = O.OracleConfig(num_workers=wl.num_workers, momentum=wl.momentum, lr=wl.lr, ns_steps=wl.ns_steps,
                         local_polar=wl.local_polar)
    st = O.init_state(specs, cfg)
    weights = [w.float().numpy().astype(np.float64) for w in wlmod.make_weights(sub)]
    signal = wlmod.make_signal(sub)
    grads = [g.float().numpy() for g in wlmod.make_grads(sub, signal, 0)]
    times = []
    for t in range(warmup + steps):
        t0 = time.perf_counter()
        weights, _ = O.step(specs, cfg, st, weights, grads)
        dt = time.perf_counter() - t0
        if t >= warmup:
            times.append(dt)
    per_sample_step = sum(times) / len(times)
    est_full = per_sample_step * c_total / c_sample
    cores = max([d.get("num_threads", 1) for d in threadpool_info()] + [1])
    return {"value": 1.0 / est_full, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(idx)} of {len(wl.params)} parameters of {wl.name} (all {wl.num_workers} workers, full "
                      f"step each), {per_sample_step:.2f} s per sample step; extrapolated to the whole workload by "
                      f"literal float64 operation count (x{c_total / c_sample:.1f})",
            "sample_seconds_per_step": per_sample_step}


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel, from the ncu
# captures summarised under profiles/; None for workloads without a capture of the current kernel.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    ("c2_resnet50", "ns_gemm_tc_kernel"): 525.7e6,   # mean of 5 Gram (230.5 MB) and 5 apply (820.8 MB) launches
}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group):
    multi-GPU times are the slowest rank's."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(ms_step, world):
    """Replicas only: every rank runs one full step per `ms_step`, so the job does `world` steps in that time."""
    return world * 1e3 / ms_step


def describe(wl):
    return {"workload": wl.name, "params": len(wl.params), "entries": wl.numel, "num_workers": wl.num_workers,
            "ns_steps": wl.ns_steps, "local_polar": bool(wl.local_polar), "momentum": wl.momentum, "lr": wl.lr,
            "weight_dtype": wl.params[0].dtype, "l2": "inputs larger than L2 (state + gradients per step > 126 MB)"}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    res = time_oracle(wl, args.steps, args.warmup, args.oracle_flops)
    ms = 1e3 / res["value"]
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": describe(wl),
            "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args, wl):
    import torch
    from paper_2605_16311_b200 import binding as B
    from paper_2605_16311_b200 import build as build_mod
    from paper_2605_16311_b200 import workloads as wlmod

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SignMuon step has no CPU fallback")
    if rank == 0:
        build_mod.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
        dist.barrier()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    B.load_library()

    opt = B.SignMuon(wl.params, wl.num_workers, momentum=wl.momentum, lr=wl.lr, ns_steps=wl.ns_steps,
                     local_polar=wl.local_polar, device=dev, host_staging=True, ns_scale=args.ns_scale,
                     power_iters=args.power_iters)
    if args.ns_scale == "spectral":     # seeded start vectors of the power iteration, reused by every step
        flat = torch.zeros(opt.power_start_size, dtype=torch.float32, device=dev)
        for p, v in enumerate(wlmod.make_power_start(wl, 0, dev)):
            if v is not None:
                off, _ = opt.power_start_segment(p)
                flat[off: off + v.numel()] = v.reshape(-1)
        opt.set_power_start(flat)
    weights = wlmod.make_weights(wl, dev)
    signal = wlmod.make_signal(wl, dev)
    n_sets = 2                                           # fresh noise per step, rotating pre-drawn sets
    grad_sets = [wlmod.make_grads(wl, signal, t, dev) for t in range(n_sets)]
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------------------------------------------------------- device-resident timing
    for t in range(args.warmup):
        opt.step(weights, grad_sets[t % n_sets], wl.lr)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(args.steps):
        opt.step(weights, grad_sets[t % n_sets], wl.lr)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    status = opt.status()
    if status != B.OK:
        raise RuntimeError(f"device status after the timed region: {status}")

    # ---------------------------------------------------------------- per-stage timing (same steps, events between stages)
    stages = [("momentum", B.STAGE_MOMENTUM), ("newton_schulz", B.STAGE_NS), ("vote_update", B.STAGE_VOTE),
              ("local_polar", B.STAGE_LOCAL_POLAR)]
    n_stage_steps = max(3, min(args.steps, 20))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)] for _ in range(n_stage_steps)]
    for t in range(n_stage_steps):
        evs[t][0].record()
        for i, (_, mask) in enumerate(stages):
            opt.step(weights, grad_sets[t % n_sets], wl.lr, stages=mask)
            evs[t][i + 1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    stage_ms = {name: statistics.mean(evs[t][i].elapsed_time(evs[t][i + 1]) for t in range(n_stage_steps))
                for i, (name, _) in enumerate(stages)}

    # ---------------------------------------------------------------- end to end with host buffers
    host_w = [w.cpu().pin_memory() for w in weights]
    host_g = [[g.cpu().pin_memory() for g in gs] for gs in grad_sets]
    h2d = sum(w.numel() * w.element_size() for w in host_w) + sum(g.numel() * g.element_size() for g in host_g[0])
    d2h = sum(w.numel() * w.element_size() for w in host_w)
    e2e_steps = 0 if args.no_e2e else max(3, min(args.steps, 30))
    for t in range(0 if args.no_e2e else 2):
        opt.step_host(host_w, host_g[t % n_sets], wl.lr)
    barrier()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for t in range(e2e_steps):
        opt.step_host(host_w, host_g[t % n_sets], wl.lr)
    h1.record()
    barrier()
    e2e_ms = h0.elapsed_time(h1) / e2e_steps if e2e_steps else float("nan")

    # ---------------------------------------------------------------- reduce over ranks
    ms_step, e2e_ms = max_over_ranks([ms_total / args.steps, e2e_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    M = wl.num_workers
    mat = [p for p in wl.params if p.kind == "matrix"]
    plain = [p for p in wl.params if p.kind == "plain"]
    gb = {"f32": 4, "bf16": 2}
    ns_flops = opt.ns_flops_per_step
    lp_frac = (1.0 / (M + 1)) if wl.local_polar else 0.0
    mom_bytes = sum(M * p.numel * (gb[p.dtype] + 4 + 4 + 2) for p in mat) + \
        sum(p.numel * (M * (gb[p.dtype] + 8) + 2 * gb[p.dtype] + M / 8 + 1 / 8) for p in plain)
    vote_bytes = sum(p.numel * (M / 8 + 1 / 8 + (2 if wl.local_polar else 2 * gb[p.dtype])) for p in mat)
    n_ns_launches = 2 * wl.ns_steps
    if args.ns_scale == "spectral":      # the power iteration reads the float32 momentum 2P + 1 more times
        mom_bytes += sum(M * p.numel * 4 * (2 * args.power_iters + 1) for p in mat)
    kernels = {}
    if stage_ms["momentum"] > 0:
        kernels["momentum+plain"] = {"ms": stage_ms["momentum"], "bound": "hbm", "algorithmic_bytes": mom_bytes,
                                     "achieved_gbs": mom_bytes / stage_ms["momentum"] / 1e6}
    ns_ms = stage_ms["newton_schulz"] + stage_ms["local_polar"]
    if ns_ms > 0 and ns_flops > 0:
        kernels["ns_gemm_tc"] = {"ms": ns_ms, "bound": "tensor", "algorithmic_flops": ns_flops,
                                 "launches": n_ns_launches * (2 if wl.local_polar else 1),
                                 "achieved_tflops": ns_flops / ns_ms / 1e9}
    if "ns_gemm_tc" in kernels:
        # the iteration's own memory traffic: per entry, worker and iteration the Gram product reads the bf16 iterate
        # (2 B), the apply product reads it again as an operand (2 B) and moves hi + lo in and out (8 B)
        ns_bytes = sum(12.0 * p.numel * wl.ns_steps * (M + (1 if wl.local_polar else 0)) for p in mat)
        kernels["ns_gemm_tc"].update({"hbm_algorithmic_bytes": ns_bytes, "hbm_achieved_gbs": ns_bytes / ns_ms / 1e6,
                                      "hbm_frac_of_measured": ns_bytes / ns_ms / 1e6 / peaks["hbm_gbs"]})
    if stage_ms["vote_update"] > 0 and vote_bytes > 0:
        kernels["vote_update"] = {"ms": stage_ms["vote_update"], "bound": "hbm", "algorithmic_bytes": vote_bytes,
                                  "achieved_gbs": vote_bytes / stage_ms["vote_update"] / 1e6}
    # dominant kernel family of the step
    dom = max(kernels, key=lambda k: kernels[k]["ms"])
    kd = kernels[dom]
    if kd["bound"] == "tensor":
        launches = kd["launches"]
        per_launch_ms = kd["ms"] / launches
        achieved = kd["achieved_tflops"]
        peak = peaks["bf16_tflops_sustained"]
        roof = {"kernel": "ns_gemm_tc_kernel", "bound": "tensor", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get((wl.name, "ns_gemm_tc_kernel")),
                "flops_per_launch": ns_flops / launches, "ms_per_launch": per_launch_ms,
                "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0}
    else:
        achieved = kd["achieved_gbs"]
        peak = peaks["hbm_gbs"]
        roof = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": None, "bytes_per_launch": kd["algorithmic_bytes"],
                "ms_per_launch": kd["ms"], "peak_source": peaks["source"] + " (copy bandwidth)",
                "frac_of_nominal_8000": achieved / 8000.0}

    cpu = None
    if not args.no_cpu_baseline:
        cpu = time_oracle(wl, 1, 0, args.cpu_baseline_flops)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}

    line = {"metric": METRIC, "value": whole_job_value(ms_step, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(describe(wl), ns_scale=args.ns_scale,
                           **({"power_iters": args.power_iters} if args.ns_scale == "spectral" else {})),
            "clocks": clocks,
            "e2e": (None if args.no_e2e else
                    {"value": whole_job_value(e2e_ms, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                     "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms}),
            "gpu_launches": opt.launches_per_step * args.steps,
            "roofline": roof, "cpu_baseline": cpu,
            "stage_ms": stage_ms, "kernels": kernels,
            "ns_tflops": ns_flops / ns_ms / 1e9 if ns_ms > 0 else None,
            "multi_gpu": "replicas only" if world > 1 else None}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(args):
    """Kernel sweep: squares and 1:4 rectangles from 512 to 8192 per side, bf16,
    M in {1..32}, K in {3, 5}; Newton-Schulz timed separately from momentum and vote+update.
    Prints one JSON line per point (this mode is not the one-line benchmark contract)."""
    import torch
    from paper_2605_16311_b200 import binding as B
    from paper_2605_16311_b200 import build as build_mod
    from paper_2605_16311_b200 import workloads as wlmod
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SignMuon step has no CPU fallback")
    build_mod.build()
    B.load_library()
    peaks = load_peaks()
    sides = [512, 1024, 2048, 4096, 8192]
    shapes = [(n, n) for n in sides] + [(512, 2048), (2048, 512), (1024, 4096), (4096, 1024), (2048, 8192), (8192, 2048)]
    workers = [int(x) for x in args.sweep_workers.split(",")]
    for (r, c) in shapes:
        for M in workers:
            for K in (3, 5):
                wl = wlmod.config5(r, c, M, K)
                opt = B.SignMuon(wl.params, M, momentum=wl.momentum, lr=wl.lr, ns_steps=K, local_polar=False,
                                 device="cuda:0")
                weights = wlmod.make_weights(wl, "cuda:0")
                signal = wlmod.make_signal(wl, "cuda:0")
                grads = wlmod.make_grads(wl, signal, 0, "cuda:0")
                for _ in range(3):
                    opt.step(weights, grads, wl.lr)
                torch.cuda.synchronize()
                reps = 5
                masks = [B.STAGE_MOMENTUM, B.STAGE_NS, B.STAGE_VOTE]
                ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
                for t in range(reps):
                    ev[t][0].record()
                    for i, mask in enumerate(masks):
                        opt.step(weights, grads, wl.lr, stages=mask)
                        ev[t][i + 1].record()
                torch.cuda.synchronize()
                if opt.status() != B.OK:
                    raise RuntimeError("device status word set during the sweep")
                ms = [statistics.median(ev[t][i].elapsed_time(ev[t][i + 1]) for t in range(reps)) for i in range(3)]
                d = r * c
                ns_flops = opt.ns_flops_per_step
                mom_bytes = M * d * (2 + 4 + 4 + 2)
                vote_bytes = d * (M / 8 + 1 / 8 + 4)
                line = {"workload": f"c5:{r}x{c}:{M}:{K}", "rows": r, "cols": c, "num_workers": M, "ns_steps": K,
                        "ns_ms": ms[1], "ns_tflops": ns_flops / ms[1] / 1e9,
                        "ns_frac_of_sustained_peak": ns_flops / ms[1] / 1e9 / peaks["bf16_tflops_sustained"],
                        "momentum_ms": ms[0], "momentum_gbs": mom_bytes / ms[0] / 1e6,
                        "vote_update_ms": ms[2], "vote_update_gbs": vote_bytes / ms[2] / 1e6,
                        "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"]}
                print(json.dumps(line), flush=True)
                opt.close()
                del opt, weights, signal, grads
                torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c2", help="c1 | c2 | c3 | c4 | c4_nolp | c5:ROWSxCOLS:M[:K]")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--oracle-flops", type=float, default=1.2e11,
                    help="float64 operation budget of one oracle sample step")
    ap.add_argument("--cpu-baseline-flops", type=float, default=2.5e12,
                    help="float64 operation budget of the oracle sample timed beside the GPU run")
    ap.add_argument("--ns-scale", default="fro", choices=["fro", "spectral"],
                    help="Alg. 4 scale: Frobenius norm (default, the benchmark configuration) or power iteration")
    ap.add_argument("--power-iters", type=int, default=2)
    ap.add_argument("--sweep", action="store_true", help="run the kernel sweep (config 5) and print one line per point")
    ap.add_argument("--sweep-workers", default="1,2,4,8,16,32")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2605_16311_b200 import workloads as wlmod
    wl = wlmod.by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
