#!/usr/bin/env python
"""Benchmark of the Muon step on B200.

    python bench.py --gpus N --steps K --warmup W [--config C] [--impl reference]

One "step" is one pass of the whole hot path (momentum / norm / cast kernel,
N Newton-Schulz iterations, fused weight update) over every matrix of the
workload.  Default workload: the MoE expert bucket (198 matrices of
2048x1408 / 1408x2048, bf16 weights and gradients, fp32 momentum), the
configuration the Newton-Schulz throughput target is quoted on.

Metric: algorithmic Newton-Schulz TFLOP/s (5 * (3 m^2 n + m^3) per matrix,
symmetric products counted once) over the whole step time.  `ms_per_step` is
the absolute step time.  `e2e` is the same metric through muon_step_host:
gradients come from pinned host memory and the updated weights go back to the
host inside the timed region.

--impl reference times the CPU fp64 oracle on a bounded sample of the same
workload (it is the only reference this method has; a baseline, not a target).

With N > 1 (torchrun) the SAME parameter set is partitioned over the ranks
(Sec. 2.3, Distributed Muon: every matrix is stepped by the one rank that owns
it) and the all-gather of the updated weights over NCCL is inside the timed
region: strong scaling.  Gradients are taken as already reduced on their owner
(the reduce-scatter of Algorithm 1's first line belongs to the backward pass
and is the same as for AdamW); --reduce-grads adds it to the timed region.
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

import torch  # noqa: E402

from paper_2502_16982_b200 import workloads as wl  # noqa: E402

METRIC = "newton_schulz_tflops"
UNIT = "TFLOP/s"
WORKLOAD_NAMES = {
    1: "cfg1: one fp32 128x256 matrix",
    2: "cfg2: dense transformer 24 layers d=2048 (168 matrices, 1.61 G params)",
    3: "cfg3: MoE expert bucket, 198 matrices of 2048x1408 / 1408x2048 (0.571 G params)",
    4: "cfg4: shape sweep, 7 single matrices",
    5: "cfg5: Moonlight-shaped full parameter set (5286 matrices, 15.3 G params)",
    6: "cfg6: the five dense scaling-law models, hidden 1536-2560, MLP [H, 2.6H] (560 matrices, 4.3 G params)",
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, taken on 64 matrices of the expert-bucket shapes; it scales with the matrix count.
NCU_CAPTURE = {"matrices": 64, "gemm_bytes_per_step": 7.915e9, "gemm_launches_per_step": 16,
               "momentum_bytes_per_launch": 2.159e9}
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        # nvidia-smi numbers physical GPUs and ignores CUDA_VISIBLE_DEVICES: the GPU is named by UUID
        self.gpu_index = gpu_id
        self.proc = None
        self.lines = []  # (arrival time, text)
        self.t_begin = self.t_end = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            # nvidia-smi needs a moment before its first line; wait for it so
            # that the samples fall inside the timed region
            t0 = time.time()
            while not self.lines and time.time() - t0 < 5.0:
                time.sleep(0.02)
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def begin(self):
        self.t_begin = time.time()

    def stop(self):
        self.t_end = time.time()
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for (t, ln) in self.lines if self.t_begin is None or self.t_begin <= t <= self.t_end + 0.1]
        if not inside:  # region shorter than one sampling period: take the nearest sample
            inside = [ln for (_, ln) in self.lines[-1:]]
        for ln in inside:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons), "gpu": str(self.gpu_index)}


def oracle_sample_time(specs, hp_dict, budget_s=20.0, max_mats=4):
    """Times the CPU oracle on one matrix per distinct shape (largest groups
    first), repeating while the budget allows.  Returns (algorithmic flops
    done, seconds, description, threads)."""
    import numpy as np
    from oracle import muon_oracle as orc

    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threads = os.cpu_count() or 1
    hp = orc.Hyper(**hp_dict)
    order = sorted(specs, key=lambda s: -s.count * s.rows * s.cols)
    flops = 0.0
    secs = 0.0
    done = []
    gen = torch.Generator().manual_seed(1234)
    shapes = order[:max_mats]
    k = 0
    while secs < budget_s and k < 64:
        sp = shapes[k % len(shapes)]
        one = wl.GroupSpec(sp.rows, sp.cols, 1, sp.w_dtype, sp.g_dtype, sp.w_std, sp.g_std, sp.lognormal_scale)
        W, G, M = wl.make_group(one, int(gen.initial_seed()) + k, "cpu")
        Wd, Gd, Md = (t[0].double().numpy() for t in (W, G, M))
        t0 = time.perf_counter()
        orc.muon_step(Wd, Gd, Md, hp)
        dt = time.perf_counter() - t0
        m, n = min(sp.rows, sp.cols), max(sp.rows, sp.cols)
        flops += hp.ns_steps * (3.0 * m * m * n + float(m) ** 3)
        secs += dt
        done.append("%dx%d" % (sp.rows, sp.cols))
        k += 1
    uniq = sorted(set(done))
    return flops, secs, "%d oracle steps on single matrices of %s" % (len(done), ", ".join(uniq)), threads


def max_over_ranks(value, dist, device):
    """MAX-reduce of a scalar over the process group (identity without one)."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(job_flops, ms_per_step):
    """Aggregate metric: the work of the whole job (all ranks together step every
    matrix of the one parameter set once) over the slowest rank's time."""
    return job_flops / (ms_per_step * 1e-3) / 1e12


def hp_dict_default():
    return dict(lr=4.2e-4, wd=0.1, mu=0.95, nesterov=True, ns_steps=5, a=3.4445, b=-4.7750, c=2.0315,
                eps=1e-7, rms_scale=0.2)


def run_reference(args, rank):
    if rank != 0:
        return
    specs = wl.config_groups(args.config)
    hp = hp_dict_default()
    times, flops_per = [], 0.0
    desc, threads = "", 1
    # each step is a bounded sample; the whole run is kept to about two minutes
    budget = min(args.ref_budget, 120.0 / max(1, args.warmup + args.steps))
    for i in range(args.warmup + args.steps):
        fl, secs, desc, threads = oracle_sample_time(specs, hp, budget_s=budget, max_mats=args.ref_mats)
        if i >= args.warmup:
            times.append(secs)
            flops_per = fl
    total = sum(times)
    value = flops_per * len(times) / total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD_NAMES[args.config], "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def gpu_uuid(dev):
    try:
        u = str(torch.cuda.get_device_properties(dev).uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        return str(dev.index)


def gemm_rooflines(prof, steps, alg_flops, dense_flops, planned, executed, peaks, clocks):
    """Roofline of the Newton-Schulz GEMM launches from per-kind event times.
    `prof`: {kind: (ms, launches)} over `steps` steps; `planned` / `executed`:
    FLOPs per step by kind (muon_plan_work)."""
    kinds = ("gram", "poly", "comb")
    gemm_ms = sum(prof[k][0] for k in kinds)
    gemm_launches = sum(prof[k][1] for k in kinds)
    if not gemm_launches:
        return None, {}
    peak = float(peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops")))
    burst = float(peaks.get("bf16_tflops", peak))
    tf = lambda flops, ms: flops * steps / (ms * 1e-3) / 1e12
    per_kind = {}
    for k in kinds:
        if prof[k][1]:
            per_kind[k] = {"planned_tflops": tf(planned[k], prof[k][0]), "executed_tflops": tf(executed[k], prof[k][0]),
                           "planned_frac_of_sustained": tf(planned[k], prof[k][0]) / peak,
                           "executed_over_planned": executed[k] / planned[k]}
    planned_all = sum(planned[k] for k in kinds)
    executed_all = sum(executed[k] for k in kinds)
    achieved = tf(alg_flops, gemm_ms)
    roof = {
        "kernel": "ns_gemm_kernel (gram + poly + comb launches)", "bound": "tensor",
        "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
        "peak_source": "%s bf16_tflops_sustained" % peaks["_source"],
        "frac_of_measured_burst": achieved / burst, "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
        "numerator": "algorithmic FLOPs of Eq. 2, ns_steps * (3 m^2 n + m^3) per matrix",
        "dense_equivalent_tflops": tf(dense_flops, gemm_ms),
        "avg_launch_ms": gemm_ms / gemm_launches, "flops_per_launch": alg_flops * steps / gemm_launches,
        # what the launch sequence asks of the tensor cores (less than algorithmic where two
        # iterations share a pass over X) and what they execute (whole tiles: padding, dropped blocks)
        "planned_tflops": tf(planned_all, gemm_ms), "frac_planned": tf(planned_all, gemm_ms) / peak,
        "planned_over_algorithmic_flops": planned_all / alg_flops,
        "executed_tflops": tf(executed_all, gemm_ms), "executed_over_planned_flops": executed_all / planned_all,
        "by_kind": per_kind, "traffic": None,
    }
    if clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        # tensor-pipe utilisation implied by the executed FLOPs at the clock sampled during the run:
        # against the nominal dense rate scaled by clock / maximum clock, and as FLOPs per clock per SM
        # against the 8192 a B200 SM retires (2.25 PFLOP/s / 148 SMs / 1.856 GHz)
        roof["tensor_util_at_sampled_clock"] = tf(executed_all, gemm_ms) / (
            NOMINAL_BF16_TFLOPS * clocks["sm_mhz"] / clocks["sm_max_mhz"])
        roof["executed_flops_per_clock_per_sm"] = tf(executed_all, gemm_ms) * 1e12 / (148 * clocks["sm_mhz"] * 1e6)
    return roof, per_kind


def run_distributed(args, rank, world, local_rank):
    """N > 1: one parameter set, partitioned over the ranks (Sec. 2.3)."""
    import torch.distributed as dist
    from paper_2502_16982_b200 import binding
    from paper_2502_16982_b200.distributed import DistributedMuon

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world == 1 and "RANK" not in os.environ:  # --distributed without torchrun: a one-rank group
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29517")
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    else:
        dist.init_process_group("nccl", device_id=dev)
    specs = wl.config_groups(args.config, args.layers)
    if args.max_count is not None:
        import dataclasses
        specs = [dataclasses.replace(s, count=min(s.count, args.max_count)) for s in specs]
    hpd = hp_dict_default()
    hpd["ns_steps"] = args.ns_steps
    hp = binding.Hyper(**hpd)
    dm = DistributedMuon([(s.rows, s.cols, s.count, s.w_dtype, s.g_dtype) for s in specs], dev, dist=dist)
    # the same weights and (already reduced) gradients on every rank: same seeds everywhere
    # (the generator calls of workloads.make_group, group by group, so that the values are the N = 1 run's)
    for gi, sp in enumerate(specs):
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 * args.config + gi)
        W = wl._randn((sp.count, sp.rows, sp.cols), sp.w_std, gen, dev, sp.w_dtype)
        for j in range(sp.count):
            dm.weights[gi][j].copy_(W[j])
        del W
        G = wl.make_grads(sp, gen, dev)
        for j in range(sp.count):
            dm.grads[gi][j].copy_(G[j])
        del G
    stream = torch.cuda.current_stream(dev)
    alg_flops, _ = wl.ns_flops(specs, hp.ns_steps)

    def barrier():
        dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        dm.step(hp, reduce_grads=args.reduce_grads)
    status, which = dm.status()
    if status != 0:
        raise SystemExit("device status %d at matrix %d during warm-up" % (status, which))
    sampler = ClockSampler(gpu_uuid(dev))
    sampler.start()
    barrier()
    sampler.begin()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    timings = []
    e0.record(stream)
    for _ in range(args.steps):
        t = {}
        dm.step(hp, reduce_grads=args.reduce_grads, timing=t)
        timings.append(t)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms_step = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    status, which = dm.status()
    if status != 0:
        raise SystemExit("device status %d at matrix %d in the timed region" % (status, which))
    compute_ms = sum(t["start"].elapsed_time(t["compute_end"]) for t in timings) / args.steps
    total_ms = sum(t["start"].elapsed_time(t["end"]) for t in timings) / args.steps
    exch_ms = sum(a.elapsed_time(b) for t in timings for a, b in t["exchanges"]) / args.steps
    exposed = max(0.0, total_ms - compute_ms)
    dist_info = {
        "ranks": world, "owned_matrices_this_rank": len(dm.owned), "matrices": sum(s.count for s in specs),
        "compute_ms_per_step": max_over_ranks(compute_ms, dist, dev),
        "exchange_ms_per_step": max_over_ranks(exch_ms, dist, dev),
        "exposed_exchange_ms_per_step": max_over_ranks(exposed, dist, dev),
        "overlapped_fraction": (1.0 - exposed / exch_ms) if exch_ms > 0 else None,
        "gather_bytes_received_per_rank": dm.gather_bytes_per_rank,
        "gather_gbs_per_rank": dm.gather_bytes_per_rank / (exch_ms * 1e-3) / 1e9 if exch_ms > 0 else None,
        "gradients": "reduce-scatter inside the timed region" if args.reduce_grads
                     else "assumed already reduced on the owner (reduce-scatter left to the backward pass)",
        "load_imbalance": max(dm.loads) / (sum(dm.loads) / world),
    }
    # end to end: this rank's gradients from pinned host memory, its updated weights back
    e2e = None
    if not args.no_e2e:
        slots = [(u, dm._slot(dm.g_flat[u], u, rank), dm._slot(dm.w_flat[u], u, rank)) for u in range(dm.n_units)]
        g_host = [g.cpu().pin_memory() for _, g, _ in slots]
        w_host = [torch.empty(w.shape, dtype=w.dtype).pin_memory() for _, _, w in slots]
        h2d = sum(t.numel() * t.element_size() for t in g_host)
        d2h = sum(t.numel() * t.element_size() for t in w_host)
        e2e_steps = max(3, min(args.steps, 5))

        def one():
            for (u, g, w), gh in zip(slots, g_host):
                g.copy_(gh, non_blocking=True)
            dm.step(hp)
            for (u, g, w), wh in zip(slots, w_host):
                wh.copy_(w, non_blocking=True)

        one()
        barrier()
        e0.record(stream)
        for _ in range(e2e_steps):
            one()
        e1.record(stream)
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), dist, dev) / e2e_steps
        h2d_all = max_over_ranks(h2d, dist, dev)
        e2e = {"value": whole_job_value(alg_flops, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "note": "bytes of rank 0; every rank moves its own slots (largest: %d B up)" % int(h2d_all)}
    launches = dm._ctx.muon_last_launch_count() * len([b for b in dm.local_bucket if b is not None]) if dm._ctx else 0
    if rank == 0:
        line = {
            "metric": METRIC, "value": whole_job_value(alg_flops, ms_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD_NAMES[args.config], "matrices": sum(s.count for s in specs),
                       "params": wl.group_params(specs), "ns_steps": hp.ns_steps,
                       "parallelism": "owner-computes dp%d, in-place NCCL all-gather of W per shape bucket" % world,
                       "l2": "inputs exceed L2", "algorithmic_tflop_per_step": alg_flops / 1e12},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches * args.steps, "distributed": dist_info,
            "roofline": None, "cpu_baseline": None,
        }
        print(json.dumps(line))
    dm.close()
    dist.destroy_process_group()


def run_aux_kernels(args):
    """Event figures for the element-wise kernels the default workload does not reach: the ld/st
    momentum kernel (gradients and momenta that TMA cannot address) and the separate weight update
    (weights that TMA cannot address, or no iteration).  Matrices of the expert shapes, every tensor
    starting one element into its buffer so that nothing is 16-byte aligned; ns_steps = 0 keeps the
    step to momentum, norm, update."""
    from paper_2502_16982_b200 import binding

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    count = args.max_count or 32
    groups, keep, elems = [], [], 0
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    for rows, cols in ((2048, 1408), (1408, 2048)):
        n = rows * cols
        ws, gs, ms = [], [], []
        for _ in range(count):
            wb = (torch.randn(n + 8, generator=gen, device=dev) * 0.02).to(torch.bfloat16)
            gb = (torch.randn(n + 8, generator=gen, device=dev) * 1e-3).to(torch.bfloat16)
            mb = torch.zeros(n + 8, dtype=torch.float32, device=dev)
            keep += [wb, gb, mb]
            ws.append(wb[1:1 + n].view(rows, cols))
            gs.append(gb[1:1 + n].view(rows, cols))
            ms.append(mb[1:1 + n].view(rows, cols))
            elems += n
        groups.append((ws, gs, ms))
    ctx = binding.MuonContext(groups)
    hpd = hp_dict_default()
    hpd["ns_steps"] = 0
    hp = binding.Hyper(**hpd)
    for _ in range(3):
        ctx.muon_step(hp)
    ctx.muon_profile_enable(True)
    steps = max(3, args.steps)
    for _ in range(steps):
        ctx.muon_step(hp)
    prof = ctx.muon_profile_read()
    ctx.muon_profile_enable(False)
    status, which = ctx.muon_status()
    if status != 0:
        raise SystemExit("device status %d at matrix %d" % (status, which))
    out = {"aux_kernels": True, "matrices": 2 * count, "elements": elems, "steps": steps,
           "peak_hbm_gbs": float(peaks["hbm_gbs"]), "peak_source": peaks["_source"]}
    for kind, name, bpe in (("momentum", "momentum_cast_kernel", 12.0), ("update", "update_from_x_kernel", 6.0)):
        ms, n = prof[kind]
        gbs = bpe * elems * steps / (ms * 1e-3) / 1e9
        out[name] = {"ms_per_launch": ms / max(1, n), "launches": n, "bytes_per_element": bpe, "achieved_gbs": gbs,
                     "frac": gbs / float(peaks["hbm_gbs"])}
    print(json.dumps(out))
    ctx.muon_destroy()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5, 6])
    ap.add_argument("--layers", type=int, default=None, help="shrink configs 2 and 5 (tests only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ns-steps", type=int, default=5, help="Newton-Schulz iterations (the paper uses 5)")
    ap.add_argument("--weights", default="config", choices=["config", "fp32", "fp32+bf16copy"],
                    help="weight dtype: the configuration's own (default), fp32 master weights, or fp32 "
                         "master weights with a bf16 copy written by the step (Sec. 2.3 keeps fp32 parameters)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-adamw", action="store_true", help="skip the AdamW (non-Muon parameters) leg")
    ap.add_argument("--reduce-grads", action="store_true",
                    help="N > 1: sum the gradients over the ranks (reduce-scatter) inside the timed region")
    ap.add_argument("--aux-kernels", action="store_true",
                    help="time the element-wise kernels of the unaligned path instead (one JSON line of their own)")
    ap.add_argument("--distributed", action="store_true",
                    help="take the partitioned (N > 1) path even with one rank")
    ap.add_argument("--max-count", type=int, default=None,
                    help="cap the matrices per group (small cases for profiler captures)")
    ap.add_argument("--ref-budget", type=float, default=12.0)
    ap.add_argument("--ref-mats", type=int, default=4)
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if args.warmup < 3:
        args.warmup = 3
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Muon step has no CPU path")
    if args.aux_kernels:
        if rank == 0:
            run_aux_kernels(args)
        return
    if world > 1 or args.distributed:
        run_distributed(args, rank, world, local_rank)
        return
    from paper_2502_16982_b200 import binding

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    specs = wl.config_groups(args.config, args.layers)
    if args.max_count is not None:
        import dataclasses
        specs = [dataclasses.replace(s, count=min(s.count, args.max_count)) for s in specs]
    if args.weights != "config":
        import dataclasses
        specs = [dataclasses.replace(s, w_dtype=torch.float32) for s in specs]
    hpd = hp_dict_default()
    hpd["ns_steps"] = args.ns_steps
    hp = binding.Hyper(**hpd)

    # Inputs: seeded, drawn on the device.
    groups, state = [], []
    for gi, sp in enumerate(specs):
        W, G, M = wl.make_group(sp, 1000 * args.config + gi, dev)
        state.append((W, G, M))
        if args.weights == "fp32+bf16copy":
            copy = torch.zeros(W.shape, dtype=torch.bfloat16, device=dev)
            state.append((copy,))  # kept alive with the rest
            groups.append((wl.views(W), wl.views(G), wl.views(M), wl.views(copy)))
        else:
            groups.append((wl.views(W), wl.views(G), wl.views(M)))
    ctx = binding.MuonContext(groups)
    stream = torch.cuda.current_stream(dev)

    def barrier():
        torch.cuda.synchronize(dev)

    alg_flops, dense_flops = wl.ns_flops(specs, hp.ns_steps)
    shape_list = [(s.rows, s.cols, s.count) for s in specs]
    planned, executed = binding.muon_plan_work(shape_list, hp.ns_steps)
    sbytes = wl.stream_bytes(specs)

    # ---- device-resident timing: the headline, with no per-launch events -------------
    for _ in range(args.warmup):
        ctx.muon_step(hp)
    status, which = ctx.muon_status()
    if status != 0:
        raise SystemExit("device status %d at matrix %d during warm-up" % (status, which))
    launches_per_step = ctx.muon_last_launch_count()
    sampler = ClockSampler(gpu_uuid(dev))
    sampler.start()
    barrier()
    sampler.begin()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        ctx.muon_step(hp)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms_step = e0.elapsed_time(e1) / args.steps
    status, which = ctx.muon_status()
    if status != 0:
        raise SystemExit("device status %d at matrix %d in the timed region" % (status, which))
    value = whole_job_value(alg_flops, ms_step)

    # ---- the same steps again with an event pair around every launch: time per kernel kind --------
    ctx.muon_profile_enable(True)
    prof_steps = args.steps
    e0.record(stream)
    for _ in range(prof_steps):
        ctx.muon_step(hp)
    e1.record(stream)
    barrier()
    ms_step_profiled = e0.elapsed_time(e1) / prof_steps
    prof = ctx.muon_profile_read()
    ctx.muon_profile_enable(False)

    # ---- end to end through muon_step_host --------------------------------------
    e2e = None
    if not args.no_e2e:
        g_host, w_host = [], []
        h2d = d2h = 0
        for sp, (W, G, M) in zip(specs, [st for st in state if len(st) == 3]):
            gh = [G[i].cpu().pin_memory() for i in range(sp.count)]
            wh = [torch.empty((sp.rows, sp.cols), dtype=sp.w_dtype).pin_memory() for _ in range(sp.count)]
            g_host.append(gh)
            w_host.append(wh)
            h2d += sum(t.numel() * t.element_size() for t in gh)
            d2h += sum(t.numel() * t.element_size() for t in wh)
        e2e_steps = max(3, min(args.steps, 5))
        ctx.muon_step_host(hp, g_host, w_host)
        barrier()
        e0.record(stream)
        for _ in range(e2e_steps):
            ctx.muon_step_host(hp, g_host, w_host)
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1) / e2e_steps
        # the copies alone, one direction at a time: what the host link of this machine gives
        n_copy = 3
        e0.record(stream)
        for _ in range(n_copy):
            for (W, G, M), gh in zip([st for st in state if len(st) == 3], g_host):
                for i, t in enumerate(gh):
                    G[i].copy_(t, non_blocking=True)
        e1.record(stream)
        barrier()
        ms_up = e0.elapsed_time(e1) / n_copy
        e0.record(stream)
        for _ in range(n_copy):
            for (W, G, M), wh in zip([st for st in state if len(st) == 3], w_host):
                for i, t in enumerate(wh):
                    t.copy_(W[i], non_blocking=True)
        e1.record(stream)
        barrier()
        ms_down = e0.elapsed_time(e1) / n_copy
        # both directions at once on two streams, no kernels: what the link gives when gradients go up
        # while weights come down, which is what every step but its first and last slice does
        side = torch.cuda.Stream(device=dev)
        e0.record(stream)
        side.wait_stream(stream)
        for _ in range(n_copy):
            for (W, G, M), gh, wh in zip([st for st in state if len(st) == 3], g_host, w_host):
                for i in range(len(gh)):
                    G[i].copy_(gh[i], non_blocking=True)
                    with torch.cuda.stream(side):
                        wh[i].copy_(W[i], non_blocking=True)
        stream.wait_stream(side)
        e1.record(stream)
        barrier()
        ms_both = e0.elapsed_time(e1) / n_copy
        floor = max(ms_step, ms_up, ms_down)
        e2e = {"value": whole_job_value(alg_flops, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "h2d_gbs_in_step": h2d / (ms_e2e * 1e-3) / 1e9, "d2h_gbs_in_step": d2h / (ms_e2e * 1e-3) / 1e9,
               "h2d_alone_ms": ms_up, "h2d_alone_gbs": h2d / (ms_up * 1e-3) / 1e9,
               "d2h_alone_ms": ms_down, "d2h_alone_gbs": d2h / (ms_down * 1e-3) / 1e9,
               "both_directions_at_once_ms": ms_both, "over_both_directions_at_once": ms_e2e / max(ms_both, ms_step),
               "over_floor": ms_e2e / floor,
               "floor": "max(device-resident step, upload alone, download alone) = %.2f ms" % floor}

    # ---- roofline of the dominant kernel -----------------------------------------
    peaks = load_peaks()
    roofline, per_kind = gemm_rooflines(prof, prof_steps, alg_flops, dense_flops, planned, executed, peaks, clocks)
    mom_ms, mom_launches = prof["momentum"]
    per_kernel = {k: {"ms_per_step": v[0] / prof_steps, "launches_per_step": v[1] / prof_steps}
                  for k, v in prof.items() if v[1]}
    for k, extra in per_kind.items():
        per_kernel[k].update(extra)
    if roofline is not None:
        roofline["timed"] = "CUDA event pairs around every launch, %d steps after the headline loop (%.3f ms per step with the events, %.3f without)" % (prof_steps, ms_step_profiled, ms_step)
        if args.config == 3 and hp.ns_steps == 5 and NCU_CAPTURE.get("gemm_bytes_per_step"):
            scale = sum(s.count for s in specs) / NCU_CAPTURE["matrices"]
            roofline["traffic"] = NCU_CAPTURE["gemm_bytes_per_step"] * scale / NCU_CAPTURE["gemm_launches_per_step"]
            roofline["traffic_note"] = "DRAM bytes per launch (average of the 16 launches of a step), scaled from a 64-matrix ncu capture"
    stream_roof = None
    if mom_launches:
        gbs = sbytes * prof_steps / (mom_ms * 1e-3) / 1e9
        stream_roof = {"kernel": "momentum_tma_kernel", "bound": "hbm", "achieved": gbs,
                       "peak": float(peaks["hbm_gbs"]), "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]),
                       "peak_source": "%s hbm_gbs" % peaks["_source"], "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                       "bytes_per_element": sbytes / wl.group_params(specs), "traffic": None,
                       "algorithmic_bytes_per_launch": sbytes / max(1, mom_launches // prof_steps)}
        if args.config == 3 and NCU_CAPTURE.get("momentum_bytes_per_launch"):
            stream_roof["traffic"] = NCU_CAPTURE["momentum_bytes_per_launch"] * sum(s.count for s in specs) / NCU_CAPTURE["matrices"]

    # ---- shape sweep: every shape of the configuration on its own ---------------------
    shapes = None
    if args.config == 4:
        shapes = []
        ctx.muon_destroy()
        for gi, sp in enumerate(specs):
            one = binding.MuonContext([groups[gi]])
            for _ in range(args.warmup):
                one.muon_step(hp)
            torch.cuda.synchronize(dev)
            e0.record(stream)
            for _ in range(args.steps):
                one.muon_step(hp)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            ms = e0.elapsed_time(e1) / args.steps
            one.muon_profile_enable(True)
            for _ in range(args.steps):
                one.muon_step(hp)
            pr = one.muon_profile_read()
            one.muon_profile_enable(False)
            g_ms = sum(pr[k][0] for k in ("gram", "poly", "comb")) / args.steps
            fl, _ = wl.ns_flops([sp], hp.ns_steps)
            pl, ex = binding.muon_plan_work([(sp.rows, sp.cols, sp.count)], hp.ns_steps)
            fl_planned, fl_executed = sum(pl.values()), sum(ex.values())
            m_, n_ = min(sp.rows, sp.cols), max(sp.rows, sp.cols)
            blocks, pairs = -(-m_ // 128), -(-(-(-m_ // 128)) // 2)
            shapes.append({"shape": "%dx%d" % (sp.rows, sp.cols), "ms_per_step": ms,
                           "launches_per_step": one.muon_last_launch_count(),
                           "step_tflops": fl / (ms * 1e-3) / 1e12,
                           "gemm_tflops": fl / (g_ms * 1e-3) / 1e12,
                           "gemm_frac_of_measured_sustained": fl / (g_ms * 1e-3) / 1e12 / float(peaks.get("bf16_tflops_sustained", 1400.0)),
                           "gemm_planned_tflops": fl_planned / (g_ms * 1e-3) / 1e12,
                           "gemm_executed_tflops": fl_executed / (g_ms * 1e-3) / 1e12,
                           "iterations_in_pairs": fl_planned < fl,
                           "row_blocks": blocks, "cta_pairs_per_column_tile": pairs})
            one.muon_destroy()
        ctx = binding.MuonContext(groups)

    # ---- AdamW for the parameters Muon does not handle: embedding-sized tensors -------
    adamw = None
    if not args.no_adamw:
        torch.cuda.empty_cache()
        shape = (163840, 2048)  # Moonlight's embedding / LM head
        ps = [torch.zeros(shape, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        gs = [torch.full(shape, 1e-3, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        ms_ = [torch.zeros(shape, dtype=torch.float32, device=dev) for _ in range(2)]
        vs = [torch.zeros(shape, dtype=torch.float32, device=dev) for _ in range(2)]
        for t in range(1, 4):
            binding.muon_adamw_step(ps, gs, ms_, vs, t, lr=4.2e-4, wd=0.1)
        torch.cuda.synchronize(dev)
        e0.record(stream)
        reps = 5
        for t in range(4, 4 + reps):
            binding.muon_adamw_step(ps, gs, ms_, vs, t, lr=4.2e-4, wd=0.1)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        a_ms = e0.elapsed_time(e1) / reps
        a_bytes = 2 * shape[0] * shape[1] * 22.0
        adamw = {"kernel": "adamw_kernel", "bound": "hbm", "workload": "2 x 163840x2048 bf16 (embedding, LM head)",
                 "ms_per_launch": a_ms, "achieved": a_bytes / (a_ms * 1e-3) / 1e9, "peak": float(peaks["hbm_gbs"]),
                 "unit": "GB/s", "frac": a_bytes / (a_ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                 "bytes_per_element": 22.0}
        del ps, gs, ms_, vs

    cpu_baseline = None
    if not args.no_cpu_baseline:
        fl, secs, desc, threads = oracle_sample_time(specs, hpd, budget_s=args.ref_budget, max_mats=args.ref_mats)
        cpu_baseline = {"value": fl / secs / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": desc, "seconds": secs}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.config], "matrices": sum(s.count for s in specs),
                   "params": wl.group_params(specs), "ns_steps": hp.ns_steps, "weights": args.weights,
                   "l2": "inputs exceed L2" if wl.group_params(specs) * 8 > 126e6 else "inputs fit L2",
                   "algorithmic_tflop_per_step": alg_flops / 1e12},
        "pct_bf16_peak_measured_sustained": 100.0 * value / float(peaks.get("bf16_tflops_sustained", 1400.0)),
        "pct_bf16_peak_nominal": 100.0 * value / NOMINAL_BF16_TFLOPS,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "roofline_stream": stream_roof, "kernels": per_kernel,
        "cpu_baseline": cpu_baseline,
    }
    if shapes is not None:
        line["shapes"] = shapes
    if adamw is not None:
        line["roofline_adamw"] = adamw
    print(json.dumps(line))
    ctx.muon_destroy()


if __name__ == "__main__":
    main()
