#!/usr/bin/env python
"""Benchmark of the fused attention forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C5] [--impl ours|reference]

A step is one pass of the whole hot path (one attn_fwd call) over one batch of synthetic input
of the named configuration.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank
runs its own batch of the same configuration (weak scaling, no data-path collective).

`--impl reference` times the fp64 CPU oracle on a bounded row sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_12355_b200 import dist as adist  # noqa: E402
from paper_2506_12355_b200 import inputs  # noqa: E402

METRIC = "attention fwd TFLOP/s at 1 B200 and % of dense FP16/BF16 tensor peak"
UNIT = "TFLOP/s"

# DRAM bytes (read + write) of one launch of the attention kernel on the default workload, from
# the ncu captures summarised under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of one launch).
NCU_TRAFFIC_BYTES = {"C5": 578620928, "C4": 380163328, "C3": 269127168, "C2": 52678912}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0.0)),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# ------------------------------------------------------------------ clocks

CLOCK_QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
REASONS = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU; stop(t0, t1) keeps the samples
    whose time stamps fall inside the timed region [t0, t1] (host wall clock, seconds)."""

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + CLOCK_QUERY,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self, t0: float, t1: float):
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=10)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        rows = []
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]),
                             [n for n, val in zip(REASONS, f[5:9]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        inside = [r for r in rows if t0 <= r[0] <= t1]
        window = "timed region"
        if not inside:   # region shorter than the sampling period: take the samples nearest to it
            mid = 0.5 * (t0 + t1)
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:3]
            window = "nearest samples"
        reasons = sorted({n for r in inside for n in r[4]})
        return {"sm_mhz": float(np.median([r[1] for r in inside])), "sm_max_mhz": float(max(r[2] for r in inside)),
                "reasons": reasons, "samples": len(inside), "window": window,
                "power_w_max": max(r[3] for r in inside)}


# ------------------------------------------------------------------ the oracle legs

def oracle_sample_rows(cfg, rows_per_head):
    step = max(1, cfg.Sq // rows_per_head)
    per = np.arange(step - 1, cfg.Sq, step, dtype=np.int64)
    return np.concatenate([bh * cfg.Sq + per for bh in range(cfg.B * cfg.H)])


def sample_flops(cfg, rows):
    i = rows % cfg.Sq
    n_vis = np.minimum(i + 1, cfg.Sk) if cfg.causal else np.full_like(i, cfg.Sk)
    return float((4.0 * n_vis * cfg.D).sum())


def time_oracle(cfg, q, k, v, rows_per_head, repeats=1):
    """Seconds per pass of the oracle over the row sample, and the sample's FLOP count."""
    from oracle import attn_oracle as orc  # the only place bench.py touches oracle/
    rows = oracle_sample_rows(cfg, rows_per_head)
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.attention_rows_16(qb, kb, vb, cfg.dtype, rows, cfg.scale, cfg.causal)
        times.append(time.perf_counter() - t0)
    return times, sample_flops(cfg, rows), len(rows), orc.num_threads()


def sample_text(cfg, n_rows, rows_per_head):
    return "%d of %d query rows (every %d-th row of every head) of %s, all their visible keys" % (
        n_rows, cfg.B * cfg.H * cfg.Sq, max(1, cfg.Sq // rows_per_head), cfg.name)


ORACLE_ROWS_PER_HEAD = {"C1": 128, "C2": 1024, "C3": 512, "C4": 256, "C5": 512}


def run_reference(args, cfg):
    rank, _, world = adist.env_world()
    if rank != 0:
        return
    q, k, v = inputs.make_config_inputs(cfg)
    # size a step so that warm-up + timed steps take about a minute: calibrate on a small sample
    cal_rph = max(1, ORACLE_ROWS_PER_HEAD[cfg.name] // 32)
    cal_t, cal_fl, _, _ = time_oracle(cfg, q, k, v, cal_rph)
    budget_s = 60.0 / max(1, args.warmup + args.steps)
    rph = int(cal_rph * budget_s / max(cal_t[0], 1e-6))
    rph = max(1, min(rph, ORACLE_ROWS_PER_HEAD[cfg.name], cfg.Sq))
    times, fl, n_rows, cores = time_oracle(cfg, q, k, v, rph, repeats=args.warmup + args.steps)
    timed = times[args.warmup:]
    sec = sum(timed) / len(timed)
    val = fl / sec / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.workload, "sample_per_step": sample_text(cfg, n_rows, rph)},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample_text(cfg, n_rows, rph)},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ our arm

def run_ours(args, cfg):
    from paper_2506_12355_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    rank, local_rank, world = adist.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()

    seed = adist.rank_seed(inputs.BASE_SEED + 1000 * cfg.index, rank)
    q, k, v = inputs.make_qkv(cfg.B, cfg.H, cfg.Sq, cfg.Sk, cfg.D, cfg.dtype, seed, cfg.sigma)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    o = torch.empty_like(qd)
    lse = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32, device=dev)
    # a buffer larger than L2, rewritten between timed steps when the inputs alone would fit in L2
    step_bytes = 4 * q.numel() * 2
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if step_bytes < (256 << 20) else None

    def step():
        api.attn_fwd(qd, kd, vd, cfg.scale, cfg.causal, out=o, lse=lse)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status after warm-up")

    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    adist.barrier()
    torch.cuda.synchronize()
    wall0 = time.time()
    for i in range(args.steps):
        if flush is not None:
            flush.fill_(i & 0xff)
        starts[i].record()
        step()
        ends[i].record()
    torch.cuda.synchronize()
    wall1 = time.time()
    adist.barrier()
    clocks = sampler.stop(wall0, wall1)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status in the timed region")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    ms_per_step_local = sum(kernel_ms) / len(kernel_ms)          # the kernel launches only
    ms_per_step = adist.reduce_scalar(ms_per_step_local, "max", dev)
    total_flops = adist.reduce_scalar(cfg.flops, "sum", dev)
    value = total_flops / (ms_per_step * 1e-3) / 1e12

    # ---- end to end: host buffers through the C ABI, copies inside the timed region ----
    qp, kp, vp = q.pin_memory(), k.pin_memory(), v.pin_memory()
    op = torch.empty_like(q).pin_memory()
    lp = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32).pin_memory()
    ws = torch.empty(api.attn_fwd_host_workspace_bytes(cfg.B, cfg.H, cfg.Sq, cfg.Sk, cfg.D), dtype=torch.uint8,
                     device=dev)
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        api.attn_fwd_host(qp, kp, vp, cfg.scale, cfg.causal, op, lp, ws)
    torch.cuda.synchronize()
    adist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        api.attn_fwd_host(qp, kp, vp, cfg.scale, cfg.causal, op, lp, ws)
    e1.record()
    torch.cuda.synchronize()
    adist.barrier()
    e2e_ms = adist.reduce_scalar(e0.elapsed_time(e1) / e2e_steps, "max", dev)
    e2e_value = total_flops / (e2e_ms * 1e-3) / 1e12
    h2d = 3 * q.numel() * 2 if cfg.Sq == cfg.Sk else (q.numel() + 2 * k.numel()) * 2
    d2h = q.numel() * 2 + lp.numel() * 4

    if rank != 0:
        return
    # ---- roofline of the dominant (only) kernel, per launch on one GPU ----
    achieved = cfg.flops / (ms_per_step_local * 1e-3) / 1e12
    roofline = {
        "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
        "frac": achieved / peaks["bf16_tflops"], "traffic": NCU_TRAFFIC_BYTES.get(cfg.name),
        "peak_source": "of %s (cuBLAS bf16 burst; fp16 has the same nominal rate)" % peaks["source"],
        "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
        "frac_of_datasheet_2250": achieved / 2250.0,
        "algorithmic_flops_per_launch": cfg.flops,
        "hbm_gbs_at_min_bytes": cfg.min_hbm_bytes / (ms_per_step_local * 1e-3) / 1e9,
        "kernel_ms_min": min(kernel_ms), "kernel_ms_median": float(np.median(kernel_ms)),
    }
    # ---- the oracle timed on this machine's host cores (bounded sample) ----
    cpu = None
    if not args.no_cpu_baseline:
        # calibrate on a small sample, then size the timed sample for roughly 15 s of CPU work
        cal = max(1, ORACLE_ROWS_PER_HEAD[cfg.name] // 8)
        cal_t, _, _, _ = time_oracle(cfg, q, k, v, cal)
        rph = int(min(cfg.Sq, max(cal, cal * 15.0 / max(cal_t[0], 1e-6))))
        times, fl, n_rows, cores = time_oracle(cfg, q, k, v, rph)
        cpu = {"value": fl / times[0] / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": sample_text(cfg, n_rows, rph), "seconds": times[0]}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == inputs.DTYPE_BF16 else "fp16", "data": "synthetic",
        "config": {"workload": cfg.workload, "per_gpu_batch": cfg.B, "global_batch": cfg.B * world,
                   "parallelism": "independent batches per GPU, no collective",
                   "l2": ("inputs+outputs %d MiB per step, larger than L2" % (step_bytes >> 20)) if flush is None
                   else "256 MiB flush buffer rewritten between timed steps"},
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": args.steps, "clocks": clocks,
        "pct_of_peak": {"measured_burst": 100 * value / world / peaks["bf16_tflops"],
                        "measured_sustained": 100 * value / world / peaks["bf16_tflops_sustained"]
                        if peaks["bf16_tflops_sustained"] else None,
                        "datasheet_2250": 100 * value / world / 2250.0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="C5", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = inputs.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
