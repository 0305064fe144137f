#!/usr/bin/env python
"""Benchmark of the fused attention forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C5] [--impl ours|reference]
                    [--kernel-only] [--no-cpu-baseline] [--no-configs] [--sustained-s SEC]
                    [--sweep grid|configs|shards|decode|bwd ...]

A step is one pass of the whole hot path (one attn_fwd call) over one batch of synthetic input of the
named configuration (default C5, the configuration the target is quoted on).  Rank 0 prints ONE JSON line:

  value / ms_per_step   K timed steps, CUDA events on the launching stream, max over ranks
  roofline              the kernel against the measured dense bf16 peak
  errors                the timed output against the fp64 oracle rows that the cpu_baseline leg computes
  configs               C1..C5, each timed as isolated launches (L2 flushed in between) with its own errors
  sustained             the same launch back to back for a few seconds, with the sampled SM clock
  backward              attn_bwd on the two causal configurations (time, TFLOP/s) and its errors on a small problem
  e2e                   host buffers through attn_fwd_host, copies inside the timed region
  cpu_baseline          the oracle timed on this machine's host cores on a bounded row sample

With --gpus N > 1 the script starts N ranks itself (torchrun) unless it already runs inside one; every rank
runs its own batch of the configuration (weak scaling, no data-path collective) and rank 0 adds
`kv_sharded_check`, a small K/V-sharded problem through dist.kv_sharded_attention.

`--impl reference` times the fp64 CPU oracle on a bounded row sample of the same workload.
`--sweep ...` prints throughput tables (markdown) instead of the JSON line.
"""
from __future__ import annotations

import argparse
import datetime
import json
import math
import os
import socket
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

# DRAM bytes (read + write) of one launch of the attention kernel, from the ncu captures summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of one launch of each configuration).
NCU_TRAFFIC_BYTES = {"C5": 574678784, "C4": 267432192, "C3": 268803584, "C2": 52238080, "C1": 173056}

O_TOL = {inputs.DTYPE_FP16: 1e-2, inputs.DTYPE_BF16: 2e-2}   # max-abs bars on O and LSE against the oracle
LSE_TOL = 1e-3


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
    """Samples nvidia-smi clocks and throttle reasons of one GPU (read only); window(t0, t1) summarises the
    samples whose time stamps fall inside [t0, t1] (host wall clock, seconds)."""

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu_index = gpu_index
        self.rows = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + CLOCK_QUERY,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            self.rows = []
            return
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
        self.rows = rows

    def window(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        inside = [r for r in self.rows if t0 <= r[0] <= t1]
        window = "timed region"
        if not inside:   # region shorter than the sampling period: take the samples nearest to it
            mid = 0.5 * (t0 + t1)
            inside = sorted(self.rows, key=lambda r: abs(r[0] - mid))[:3]
            window = "nearest samples"
        reasons = sorted({n for r in inside for n in r[4]})
        return {"sm_mhz": float(np.median([r[1] for r in inside])), "sm_max_mhz": float(max(r[2] for r in inside)),
                "reasons": reasons, "samples": len(inside), "window": window,
                "power_w_max": max(r[3] for r in inside)}


# ------------------------------------------------------------------ the oracle legs

def oracle_sample_rows(cfg, rows_per_head):
    """Every (Sq / rows_per_head)-th row of every (batch, head), ending on the head's last row."""
    step = max(1, cfg.Sq // rows_per_head)
    per = np.arange(step - 1, cfg.Sq, step, dtype=np.int64)
    return np.concatenate([bh * cfg.Sq + per for bh in range(cfg.B * cfg.H)])


def sample_flops(cfg, rows):
    i = rows % cfg.Sq
    n_vis = np.minimum(i + 1, cfg.Sk) if cfg.causal else np.full_like(i, cfg.Sk)
    return float((4.0 * n_vis * cfg.D).sum())


def run_oracle(cfg, q, k, v, rows_per_head, repeats=1):
    """The oracle over the row sample: seconds per pass, the sample (rows, FLOPs), the threads it used and the
    fp64 results of the last pass."""
    from oracle import attn_oracle as orc  # bench.py touches oracle/ only in the functions of this section
    rows = oracle_sample_rows(cfg, rows_per_head)
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        o_ref, lse_ref = orc.attention_rows_16(qb, kb, vb, cfg.dtype, rows, cfg.scale, cfg.causal)
        times.append(time.perf_counter() - t0)
    return {"times": times, "flops": sample_flops(cfg, rows), "rows": rows, "cores": orc.num_threads(),
            "o_ref": o_ref, "lse_ref": lse_ref, "rows_per_head": rows_per_head}


def sample_text(cfg, n_rows, rows_per_head):
    return "%d of %d query rows (every %d-th row of every head) of %s, all their visible keys" % (
        n_rows, cfg.B * cfg.H * cfg.Sq, max(1, cfg.Sq // rows_per_head), cfg.name)


def errors_against(cfg, o_cpu, lse_cpu, orun):
    """Error figures of a GPU result (CPU tensors of the whole problem) on the oracle's row sample."""
    rows = orun["rows"]
    idx = torch.from_numpy(rows)
    got_o = o_cpu.reshape(-1, cfg.D)[idx].to(torch.float64).numpy()
    got_l = lse_cpu.reshape(-1)[idx].to(torch.float64).numpy()
    err = np.abs(got_o - orun["o_ref"])
    row_max = err.max(axis=1)
    worst = int(row_max.argmax())
    ref_row_max = np.abs(orun["o_ref"]).max(axis=1)
    rel = row_max / np.maximum(ref_row_max, 1e-30)
    e = {"max_abs_o": float(row_max.max()), "max_abs_lse": float(np.abs(got_l - orun["lse_ref"]).max()),
         "max_rel_o": float(rel.max()),   # worst row: max |dO| of the row over max |O| of the row
         "rms_o": float(math.sqrt((err ** 2).mean() / max((orun["o_ref"] ** 2).mean(), 1e-300))),
         "argmax_row": int(rows[worst]), "rows_checked": int(rows.size),
         "tol_o": O_TOL[cfg.dtype], "tol_lse": LSE_TOL}
    e["within_tolerance"] = bool(e["max_abs_o"] <= e["tol_o"] and e["max_abs_lse"] <= e["tol_lse"]
                                 and np.isfinite(got_o).all())
    return e


def oracle_rows_for_budget(cfg, gflop_budget):
    """Rows per head whose oracle pass costs about `gflop_budget` GFLOP (all rows when the problem is smaller),
    never fewer than one row per 128-row Q tile."""
    rph = int(cfg.Sq * min(1.0, gflop_budget * 1e9 / cfg.flops))
    return max(min(cfg.Sq, (cfg.Sq + 127) // 128), min(cfg.Sq, rph))


ORACLE_ROWS_PER_HEAD = {"C1": 128, "C2": 1024, "C3": 512, "C4": 256, "C5": 512}


def run_reference(args, cfg):
    rank, _, world = adist.env_world()
    if rank != 0:
        return 0
    q, k, v = inputs.make_config_inputs(cfg)
    # size a step so that warm-up + timed steps take about a minute: calibrate on a small sample
    cal_rph = max(1, ORACLE_ROWS_PER_HEAD[cfg.name] // 32)
    cal = run_oracle(cfg, q, k, v, cal_rph)
    budget_s = 60.0 / max(1, args.warmup + args.steps)
    rph = int(cal_rph * budget_s / max(cal["times"][0], 1e-6))
    rph = max(1, min(rph, ORACLE_ROWS_PER_HEAD[cfg.name], cfg.Sq))
    run = run_oracle(cfg, q, k, v, rph, repeats=args.warmup + args.steps)
    timed = run["times"][args.warmup:]
    sec = sum(timed) / len(timed)
    val = run["flops"] / sec / 1e12
    text = sample_text(cfg, run["rows"].size, rph)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.workload, "sample_per_step": text},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": run["cores"], "kind": "oracle", "sample": text},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------ timing helpers

def time_isolated(fn, flush, launches, warmup=10):
    """CUDA-event time (ms) of every one of `launches` isolated calls of fn on the current stream, a buffer larger
    than L2 rewritten before each one."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    a = [torch.cuda.Event(enable_timing=True) for _ in range(launches)]
    b = [torch.cuda.Event(enable_timing=True) for _ in range(launches)]
    for i in range(launches):
        flush.fill_(i & 0xff)
        a[i].record()
        fn()
        b[i].record()
    torch.cuda.synchronize()
    return [x.elapsed_time(y) for x, y in zip(a, b)]


class Problem:
    """Device tensors of one configuration (inputs from the seeded recipe) and its launch."""

    def __init__(self, api, cfg, dev, seed=None):
        self.api, self.cfg, self.dev = api, cfg, dev
        seed = inputs.BASE_SEED + 1000 * cfg.index if seed is None else seed
        self.q, self.k, self.v = inputs.make_qkv(cfg.B, cfg.H, cfg.Sq, cfg.Sk, cfg.D, cfg.dtype, seed, cfg.sigma)
        self.qd, self.kd, self.vd = self.q.to(dev), self.k.to(dev), self.v.to(dev)
        self.o = torch.empty_like(self.qd)
        self.lse = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32, device=dev)

    def step(self):
        self.api.attn_fwd(self.qd, self.kd, self.vd, self.cfg.scale, self.cfg.causal, out=self.o, lse=self.lse)

    def poison(self):
        self.o.fill_(float("nan"))
        self.lse.fill_(float("nan"))


def host_enqueue_us(api, prob, calls):
    """Host time of one attn_fwd call through the C ABI (arguments prepared once; validation, tensor maps and
    the launch), while the device works through the queue."""
    cfg = prob.cfg
    fn = api.load().attn_fwd
    a = (prob.qd.data_ptr(), prob.kd.data_ptr(), prob.vd.data_ptr(), prob.o.data_ptr(), prob.lse.data_ptr(), cfg.B, cfg.H,
         cfg.Sq, cfg.Sk, cfg.D, cfg.scale, int(cfg.causal), cfg.dtype, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(calls):
        fn(*a)
    t1 = time.perf_counter()
    torch.cuda.synchronize()
    return (t1 - t0) / calls * 1e6


def graph_replay_us(prob, flush, launches):
    """Median device time of the launch replayed from a CUDA graph (isolated, L2 flushed)."""
    st = torch.cuda.Stream(device=prob.dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            prob.api.attn_fwd(prob.qd, prob.kd, prob.vd, prob.cfg.scale, prob.cfg.causal, out=prob.o, lse=prob.lse,
                              stream=st)
    torch.cuda.synchronize()
    return float(np.median(time_isolated(g.replay, flush, launches, warmup=3))) * 1e3


def config_block(api, dev, peaks, flush, headline, headline_errors, with_errors):
    """C1..C5 as isolated launches (L2 flushed in between): time, throughput, bandwidth at the algorithmic bytes
    and the errors of that output against the oracle."""
    out = {}
    for name in sorted(inputs.CONFIGS):
        cfg = inputs.CONFIGS[name]
        prob = headline if name == headline.cfg.name else Problem(api, cfg, dev)
        launches = 200 if name in ("C1", "C2") else 50
        prob.poison()
        ms = time_isolated(prob.step, flush, launches)
        med, mn = float(np.median(ms)), min(ms)
        entry = {"workload": cfg.workload, "launches": launches, "us_median": med * 1e3, "us_min": mn * 1e3,
                 "tflops": cfg.flops / med / 1e9, "frac_of_burst": cfg.flops / med / 1e9 / peaks["bf16_tflops"],
                 "gbs_at_min_bytes": cfg.min_hbm_bytes / med / 1e6,
                 "frac_of_hbm_peak": cfg.min_hbm_bytes / med / 1e6 / peaks["hbm_gbs"],
                 "ncu_dram_bytes": NCU_TRAFFIC_BYTES.get(name), "min_hbm_bytes": cfg.min_hbm_bytes,
                 "host_us_per_call": host_enqueue_us(api, prob, 200 if name in ("C1", "C2") else 20)}
        if name in ("C1", "C2", "C3"):   # launch-latency territory: the same launch replayed from a CUDA graph
            entry["us_graph_replay_median"] = graph_replay_us(prob, flush, 50)
        if with_errors:
            if name == headline.cfg.name and headline_errors is not None:
                entry["errors"] = headline_errors
            else:
                orun = run_oracle(cfg, prob.q, prob.k, prob.v, oracle_rows_for_budget(cfg, 120.0))
                entry["errors"] = errors_against(cfg, prob.o.cpu(), prob.lse.cpu(), orun)
        out[name] = entry
        if prob is not headline:
            del prob
    return out


def sustained_block(prob, sampler_index, peaks, seconds, ms_guess):
    """The same launch back to back for `seconds`: mean time per launch with the SM clock sampled meanwhile."""
    n = max(20, int(seconds * 1e3 / max(ms_guess, 1e-3)))
    sampler = ClockSampler(sampler_index)
    sampler.start()
    time.sleep(0.1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    w0 = time.time()
    e0.record()
    for _ in range(n):
        prob.step()
    e1.record()
    torch.cuda.synchronize()
    w1 = time.time()
    sampler.stop()
    # the first tenth of the window is the ramp from idle clocks; summarise the clocks of the rest
    clocks = sampler.window(w0 + 0.1 * (w1 - w0), w1)
    ms = e0.elapsed_time(e1) / n
    tf = prob.cfg.flops / ms / 1e9
    return {"seconds": (w1 - w0), "launches": n, "ms_mean": ms, "tflops": tf,
            "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
            "frac_of_burst_peak": tf / peaks["bf16_tflops"],
            "sm_mhz_median": clocks.get("sm_mhz"), "ms_x_mhz": ms * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
            "power_w_max": clocks.get("power_w_max"), "reasons": clocks.get("reasons"), "clock_samples": clocks.get("samples")}


def backward_block(api, dev, peaks, flush, with_errors):
    """The backward pass (attn_bwd: row sums, dQ pass, dK/dV pass) on the two causal bf16 configurations, timed as
    isolated calls; FLOPs counted as 2.5 x the forward count (five tile products, of which the two passes execute
    seven).  Errors: a small problem against the oracle's fp64 gradients."""
    out = {"flops_counted": "2.5 x forward (S, dP, dV, dQ, dK); the kernels execute 3.5 x (S and dP once per pass)"}
    for name in ("C3", "C5"):
        cfg = inputs.CONFIGS[name]
        prob = Problem(api, cfg, dev)
        prob.step()
        dout = inputs.randn16((cfg.B, cfg.H, cfg.Sq, cfg.D), inputs.BASE_SEED + 1000 * cfg.index + 3, cfg.dtype).to(dev)
        dq, dk, dv = torch.empty_like(prob.qd), torch.empty_like(prob.kd), torch.empty_like(prob.vd)
        ws = torch.empty(api.attn_bwd_workspace_bytes(cfg.B, cfg.H, cfg.Sq), dtype=torch.uint8, device=dev)
        ms = time_isolated(lambda: api.attn_bwd(prob.qd, prob.kd, prob.vd, prob.o, prob.lse, dout, cfg.scale, cfg.causal,
                                                dq=dq, dk=dk, dv=dv, workspace=ws), flush, 20, warmup=3)
        med = float(np.median(ms))
        tf = 2.5 * cfg.flops / med / 1e9
        out[name] = {"workload": cfg.workload.replace("fwd", "bwd"), "ms_median": med, "ms_min": min(ms), "tflops": tf,
                     "frac_of_burst": tf / peaks["bf16_tflops"], "gpu_launches_per_call": 3}
        del prob, dout, dq, dk, dv, ws
    if with_errors:
        from oracle import attn_oracle as orc   # oracle leg: gradients of a small problem
        B, H, S, D, dt = 1, 4, 1024, 128, inputs.DTYPE_BF16
        q, k, v = inputs.make_qkv(B, H, S, S, D, dt, inputs.BASE_SEED + 555)
        dout = inputs.randn16((B, H, S, D), inputs.BASE_SEED + 558, dt)
        scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
        qd, kd, vd, dd = q.to(dev), k.to(dev), v.to(dev), dout.to(dev)
        o, lse = api.attn_fwd(qd, kd, vd, scale, True)
        got = api.attn_bwd(qd, kd, vd, o, lse, dd, scale, True)
        ref = orc.attention_bwd(*(orc.widen(inputs.bits(t), dt) for t in (q, k, v, dout)), scale, True)
        e = {"problem": "causal bf16 B=1 H=4 S=1024 D=128"}
        for nm, g, r in zip(("dq", "dk", "dv"), got, ref):
            err = np.abs(g.cpu().double().numpy() - r)
            e[nm] = {"max_abs": float(err.max()), "rms_rel": float(math.sqrt((err ** 2).mean() / (r ** 2).mean())),
                     "ref_rms": float(math.sqrt((r ** 2).mean()))}
        out["errors"] = e
    return out


def kv_sharded_check(api, dev, rank, world):
    """A small K/V-sharded problem through dist.kv_sharded_attention with both exchange forms; rank 0 compares
    the merged result with the oracle (max-abs errors).  Every rank takes the same branches."""
    B, H, S, D, dt, causal = 1, 4, 2048, 128, inputs.DTYPE_BF16, True
    q, k, v = inputs.make_qkv(B, H, S, S, D, dt, seed=inputs.BASE_SEED + 77)
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    b, e = adist.shard_keys(S, world, rank)
    qd = q.to(dev)
    ks, vs = k[:, :, b:e].contiguous().to(dev), v[:, :, b:e].contiguous().to(dev)
    peer_ok = all(torch.cuda.can_device_access_peer(i, j) for i in range(world) for j in range(world) if i != j)
    try:
        import torch.distributed._symmetric_memory  # noqa: F401
    except ImportError:
        peer_ok = False
    res = {"problem": "causal bf16 B=1 H=4 S=2048 D=128, keys split over %d ranks" % world}
    ref = None
    for exchange in ("nccl", "peer"):
        if exchange == "peer" and not peer_ok:
            res[exchange] = "unavailable: no peer access between all GPUs or no symmetric memory in this torch"
            continue
        o, lse = adist.kv_sharded_attention(qd, ks, vs, scale, causal, b, exchange=exchange)
        torch.cuda.synchronize()
        adist.barrier()
        if rank == 0:
            if ref is None:
                from oracle import attn_oracle as orc
                rows = np.arange(B * H * S, dtype=np.int64)
                ref = orc.attention_rows_16(inputs.bits(q), inputs.bits(k), inputs.bits(v), dt, rows, scale, causal)
            res[exchange] = {"max_abs_o": float(np.abs(o.cpu().double().numpy().reshape(-1, D) - ref[0]).max()),
                             "max_abs_lse": float(np.abs(lse.cpu().double().numpy().reshape(-1) - ref[1]).max())}
    return res


# ------------------------------------------------------------------ our arm

def run_ours(args, cfg):
    from paper_2506_12355_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    rank, local_rank, world = adist.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    warmup = max(args.warmup, 3)

    prob = Problem(api, cfg, dev, seed=adist.rank_seed(inputs.BASE_SEED + 1000 * cfg.index, rank))
    q, k, v = prob.q, prob.k, prob.v
    # a buffer larger than L2, rewritten between timed steps when the inputs alone would fit in L2
    step_bytes = 4 * q.numel() * 2
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_headline = step_bytes < (256 << 20)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(warmup):
        prob.step()
    torch.cuda.synchronize()
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status after warm-up")
    prob.poison()

    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    adist.barrier()
    torch.cuda.synchronize()
    wall0 = time.time()
    for i in range(args.steps):
        if flush_headline:
            flush.fill_(i & 0xff)
        starts[i].record()
        prob.step()
        ends[i].record()
    torch.cuda.synchronize()
    wall1 = time.time()
    adist.barrier()
    sampler.stop()
    clocks = sampler.window(wall0, wall1)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status in the timed region")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    ms_per_step_local = sum(kernel_ms) / len(kernel_ms)          # the kernel launches only
    ms_per_step = adist.reduce_scalar(ms_per_step_local, "max", dev)
    total_flops = adist.reduce_scalar(cfg.flops, "sum", dev)
    value = total_flops / (ms_per_step * 1e-3) / 1e12
    o_timed, lse_timed = prob.o.cpu(), prob.lse.cpu()            # the output of the last timed step

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
    if args.kernel_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "warmup": warmup, "ms_per_step": ms_per_step, "config": {"workload": cfg.workload},
                              "roofline": roofline, "gpu_launches": args.steps, "clocks": clocks,
                              "note": "kernel-only run (profiling helper): no e2e, errors, configs or cpu_baseline"}),
                  flush=True)
        return 0

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
    del ws

    kv_check = kv_sharded_check(api, dev, rank, world) if world > 1 else None
    if rank != 0:
        return 0

    # ---- single GPU only: the oracle on this machine's host cores, the errors of the timed output against it,
    # every configuration as isolated launches, and the sustained run ----
    cpu = errors = configs = sustained = backward = None
    if world == 1 and not args.no_cpu_baseline:
        # calibrate on a small sample, then size the timed sample for roughly 15 s of CPU work
        cal_rph = max(1, ORACLE_ROWS_PER_HEAD[cfg.name] // 8)
        cal = run_oracle(cfg, q, k, v, cal_rph)
        rph = int(min(cfg.Sq, max(cal_rph, cal_rph * 15.0 / max(cal["times"][0], 1e-6))))
        orun = run_oracle(cfg, q, k, v, rph)
        text = sample_text(cfg, orun["rows"].size, rph)
        cpu = {"value": orun["flops"] / orun["times"][0] / 1e12, "unit": UNIT, "cores": orun["cores"], "kind": "oracle",
               "sample": text, "seconds": orun["times"][0]}
        errors = errors_against(cfg, o_timed, lse_timed, orun)
        errors["sample"] = text
        del orun
    if world == 1 and not args.no_configs:
        configs = config_block(api, dev, peaks, flush, prob, errors, with_errors=not args.no_cpu_baseline)
    if world == 1 and args.sustained_s > 0:
        sustained = sustained_block(prob, local_rank, peaks, args.sustained_s, ms_per_step_local)
    if world == 1 and not args.no_configs:
        backward = backward_block(api, dev, peaks, flush, with_errors=not args.no_cpu_baseline)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status after the timed region")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == inputs.DTYPE_BF16 else "fp16", "data": "synthetic",
        "config": {"workload": cfg.workload, "per_gpu_batch": cfg.B, "global_batch": cfg.B * world,
                   "parallelism": "independent batches per GPU, no collective",
                   "l2": ("inputs+outputs %d MiB per step, larger than L2" % (step_bytes >> 20)) if not flush_headline
                   else "256 MiB flush buffer rewritten between timed steps"},
        "roofline": roofline, "errors": errors, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": args.steps, "clocks": clocks,
        "pct_of_peak": {"measured_burst": 100 * value / world / peaks["bf16_tflops"],
                        "measured_sustained": 100 * value / world / peaks["bf16_tflops_sustained"]
                        if peaks["bf16_tflops_sustained"] else None,
                        "datasheet_2250": 100 * value / world / 2250.0},
        "sustained": sustained, "configs": configs, "backward": backward,
    }
    if kv_check is not None:
        line["kv_sharded_check"] = kv_check
    print(json.dumps(line), flush=True)
    bad = [n for n, c in (configs or {}).items() if c.get("errors") and not c["errors"]["within_tolerance"]]
    if errors is not None and not errors["within_tolerance"]:
        bad.append(cfg.name + " (timed output)")
    if bad:
        print("bench.py: output outside the tolerance against the oracle: %s" % ", ".join(bad), file=sys.stderr)
        return 3
    return 0


def run_stub(args):
    """The timing protocol with an empty CPU step on gloo ranks: exercises the launcher and the cross-rank
    reductions where there is no GPU.  It measures nothing and says so."""
    rank, local_rank, world = adist.init("gloo")
    adist.barrier()
    ms = adist.reduce_scalar(float(rank + 1), "max", "cpu")
    units = adist.reduce_scalar(1.0, "sum", "cpu")
    adist.barrier()
    if rank == 0:
        print(json.dumps({"impl": "stub", "n_gpus": world, "value": None, "ranks_seen": units, "max_over_ranks": ms,
                          "note": "launcher self-test on CPU, no attention computed"}), flush=True)
    return 0


# ------------------------------------------------------------------ launcher

def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n: int, argv) -> int:
    """Re-runs this script as n ranks (one per GPU) under torch.distributed.run on this node."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")          # keeps NCCL's communicator log (rings, NVLS) in the output
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    return subprocess.call(cmd, env=env)


# ------------------------------------------------------------------ sweeps (markdown tables, not the JSON line)

def sweep_time(fn, flush, iters):
    ts = sorted(time_isolated(fn, flush, iters, warmup=3))
    return ts[len(ts) // 2]


def sweep_shards(api, args, dev, flush):
    n, H, D, dt = args.shards, 32, 128, inputs.DTYPE_BF16
    print("| sequence | unsharded ms | %d partial launches ms | merge us | merge GB/s | sharded / unsharded |" % n)
    print("|---|---|---|---|---|---|")
    for S in ([args.seq] if args.seq else [4096, 16384]):
        q = inputs.randn16((1, H, S, D), 1, dt).to(dev)
        k = inputs.randn16((1, H, S, D), 2, dt).to(dev)
        v = inputs.randn16((1, H, S, D), 3, dt).to(dev)
        o = torch.empty_like(q)
        lse = torch.empty((1, H, S), dtype=torch.float32, device=dev)
        o_parts = torch.empty((n, 1, H, S, D), dtype=q.dtype, device=dev)
        l_parts = torch.empty((n, 1, H, S), dtype=torch.float32, device=dev)
        bounds = [S * i // n // 128 * 128 for i in range(n)] + [S]
        ks = [k[:, :, bounds[i]:bounds[i + 1]].contiguous() for i in range(n)]
        vs = [v[:, :, bounds[i]:bounds[i + 1]].contiguous() for i in range(n)]
        scale = D ** -0.5

        def partials():
            for i in range(n):
                api.attn_fwd_partial(q, ks[i], vs[i], scale, True, bounds[i], out=o_parts[i], lse=l_parts[i])

        t_full = sweep_time(lambda: api.attn_fwd(q, k, v, scale, True, out=o, lse=lse), flush, args.iters)
        t_part = sweep_time(partials, flush, args.iters)
        t_merge = sweep_time(lambda: api.attn_combine(o_parts, l_parts, out=o, lse=lse), flush, args.iters)
        moved = (n + 1) * H * S * (D * 2 + 4)
        print("| %d | %.3f | %.3f | %.1f | %.0f | %.2f |" % (S, t_full, t_part, t_merge * 1e3, moved / t_merge / 1e6,
                                                       (t_part + t_merge) / t_full), flush=True)


def sweep_decode(api, args, dev, flush):
    D, dt = 128, inputs.DTYPE_BF16
    splits = [1, 2, 4, 8, 16, 32]
    print("| batch x heads (K/V heads) x keys | K+V MB | " + " | ".join("%d ranges: us (GB/s)" % n for n in splits) + " |")
    print("|---|---|" + "---|" * len(splits))
    for (B, H, Hkv, Sk) in ((1, 32, 8, 16384), (1, 32, 8, 65536), (1, 32, 32, 65536), (8, 32, 8, 16384)):
        if args.seq and Sk != args.seq:
            continue
        q = inputs.randn16((B, H, 1, D), 1, dt).to(dev)
        k = inputs.randn16((B, Hkv, Sk, D), 2, dt).to(dev)
        v = inputs.randn16((B, Hkv, Sk, D), 3, dt).to(dev)
        o = torch.empty_like(q)
        lse = torch.empty((B, H, 1), dtype=torch.float32, device=dev)
        ws = torch.empty(api.attn_fwd_splitkv_workspace_bytes(B, H, 1, D, max(splits)), dtype=torch.uint8, device=dev)
        kv_bytes = 2.0 * B * Hkv * Sk * D * 2
        cells = []
        for n in splits:
            ms = sweep_time(lambda: api.attn_fwd_splitkv(q, k, v, D ** -0.5, False, n, workspace=ws, out=o, lse=lse),
                            flush, args.iters)
            cells.append("%.0f (%.0f)" % (ms * 1e3, kv_bytes / ms / 1e6))
        if args.graph:
            # the same calls replayed from a CUDA graph (launch overhead off the device timeline)
            cells_g = []
            for n in splits:
                st = torch.cuda.Stream(device=dev)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.stream(st):
                    with torch.cuda.graph(g, stream=st):
                        api.attn_fwd_splitkv(q, k, v, D ** -0.5, False, n, workspace=ws, out=o, lse=lse, stream=st)
                ms = sweep_time(g.replay, flush, args.iters)
                cells_g.append("%.0f (%.0f)" % (ms * 1e3, kv_bytes / ms / 1e6))
        print("| %d x %d (%d) x %d | %.0f | %s |" % (B, H, Hkv, Sk, kv_bytes / 1e6, " | ".join(cells)), flush=True)
        if args.graph:
            print("| (graph replay) | | %s |" % " | ".join(cells_g), flush=True)
        del q, k, v, o, lse, ws


def sweep_configs(api, args, dev, flush):
    print("| config | time | TFLOP/s | GB/s at algorithmic bytes |")
    print("|---|---|---|---|")
    for name in sorted(inputs.CONFIGS):
        prob = Problem(api, inputs.CONFIGS[name], dev)
        ms = sweep_time(prob.step, flush, max(args.iters, 30))
        print("| %s | %.1f us | %.1f | %.0f |" % (prob.cfg.workload, ms * 1e3, prob.cfg.flops / ms / 1e9,
                                                 prob.cfg.min_hbm_bytes / ms / 1e6), flush=True)
        del prob


def sweep_grid(api, args, dev, flush):
    """The benchmark grid of the paper's Section 4.1: sequence 512..16k at 16k tokens per batch, hidden size 2048
    (32 heads of dim 64 or 16 of dim 128), with and without the causal mask; in addition head dim 256 (8 heads)
    and the 192/128 head shape (16 heads); --dtype fp8: the FP8 case of Section 4.4 (16 heads of dim 128, E4M3).
    FLOPs as in the paper: 4 seq^2 head_dim heads per batch element, halved for causal rows."""
    dt = inputs.DTYPE_BF16 if args.dtype == "bf16" else inputs.DTYPE_FP16
    seqs = [512, 1024, 2048, 4096, 8192, 16384]
    if args.seq:
        if args.seq not in seqs:
            raise SystemExit("--seq must be one of %s" % seqs)
        seqs = [args.seq]
    shapes = [("D=64", 32, 64, 64), ("D=128", 16, 128, 128), ("D=256", 8, 256, 256), ("Dqk=192 Dv=128", 16, 192, 128)]
    if args.dtype == "fp8":
        shapes = [("D=128 E4M3", 16, 128, 128)]
    print("| heads x dims | mask | " + " | ".join(str(s) for s in seqs) + " |")
    print("|---|---|" + "---|" * len(seqs))
    for name, H, Dqk, Dv in shapes:
        Hkv = args.gqa if args.gqa and H % args.gqa == 0 else H
        for causal in (True, False):
            cells = []
            for S in seqs:
                B = 16384 // S
                if args.dtype == "fp8":
                    q = inputs.randn8((B, H, S, Dqk), 1).to(dev)
                    k = inputs.randn8((B, Hkv, S, Dqk), 2).to(dev)
                    v = inputs.randn8((B, Hkv, S, Dv), 3).to(dev)
                    o = torch.empty((B, H, S, Dv), dtype=torch.bfloat16, device=dev)
                else:
                    q = inputs.randn16((B, H, S, Dqk), 1, dt).to(dev)
                    k = inputs.randn16((B, Hkv, S, Dqk), 2, dt).to(dev)
                    v = inputs.randn16((B, Hkv, S, Dv), 3, dt).to(dev)
                    o = torch.empty((B, H, S, Dv), dtype=q.dtype, device=dev)
                lse = torch.empty((B, H, S), dtype=torch.float32, device=dev)
                scale = Dqk ** -0.5
                if args.dtype == "fp8":
                    fn = lambda: api.attn_fwd_fp8(q, k, v, scale, 1.0, 1.0, 1.0, causal, out=o, lse=lse)  # noqa: E731
                elif Dqk == Dv:
                    fn = lambda: api.attn_fwd_gqa(q, k, v, scale, causal, out=o, lse=lse)  # noqa: E731
                else:
                    fn = lambda: api.attn_fwd_qkv_dims(q, k, v, scale, causal, out=o, lse=lse)  # noqa: E731
                ms = sweep_time(fn, flush, args.iters)
                flops = 2.0 * B * H * S * S * (Dqk + Dv) / (2 if causal else 1)
                cells.append("%.0f" % (flops / ms / 1e9))
                del q, k, v, o, lse
            print("| %d x %s%s | %s | %s |" % (H, name, "" if Hkv == H else " (Hkv=%d)" % Hkv,
                                              "causal" if causal else "none", " | ".join(cells)), flush=True)


def sweep_bwd(api, args, dev, flush):
    """The backward pass (attn_bwd: row sums + dQ pass + dK/dV pass) on the grid of sweep_grid for head dims 64 and
    128; FLOPs counted as 2.5 x the forward count (five tile products: S, dP, dV, dQ, dK; the kernels execute
    seven, S and dP once per pass)."""
    dt = inputs.DTYPE_BF16 if args.dtype == "bf16" else inputs.DTYPE_FP16
    seqs = [args.seq] if args.seq else [512, 1024, 2048, 4096, 8192, 16384]
    print("| heads x dim | mask | " + " | ".join("%d: ms (TFLOP/s)" % s for s in seqs) + " |")
    print("|---|---|" + "---|" * len(seqs))
    for H, D in ((32, 64), (16, 128)):
        for causal in (True, False):
            cells = []
            for S in seqs:
                B = max(1, 16384 // S)
                q, k, v = (t.to(dev) for t in inputs.make_qkv(B, H, S, S, D, dt, 1))
                dout = inputs.randn16((B, H, S, D), 4, dt).to(dev)
                scale = D ** -0.5
                o, lse = api.attn_fwd(q, k, v, scale, causal)
                dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
                ws = torch.empty(api.attn_bwd_workspace_bytes(B, H, S), dtype=torch.uint8, device=dev)
                ms = sweep_time(lambda: api.attn_bwd(q, k, v, o, lse, dout, scale, causal, dq=dq, dk=dk, dv=dv, workspace=ws),
                                flush, args.iters)
                flops = 2.5 * 4.0 * B * H * S * S * D / (2 if causal else 1)
                cells.append("%.3f (%.0f)" % (ms, flops / ms / 1e9))
                del q, k, v, dout, o, lse, dq, dk, dv, ws
            print("| %d x %d | %s | %s |" % (H, D, "causal" if causal else "none", " | ".join(cells)), flush=True)


def run_sweep(args):
    from paper_2506_12355_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    dev = torch.device("cuda:0")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    {"grid": sweep_grid, "configs": sweep_configs, "shards": sweep_shards, "decode": sweep_decode, "bwd": sweep_bwd}[args.sweep](
        api, args, dev, flush)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status")
    return 0


def main(argv=None):
    argv = sys.argv[1:] if argv is None else list(argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="C5", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "stub"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle legs (cpu_baseline and errors)")
    ap.add_argument("--no-configs", action="store_true", help="skip the C1..C5 block")
    ap.add_argument("--sustained-s", type=float, default=2.0, help="length of the back-to-back run (0: skip)")
    ap.add_argument("--kernel-only", action="store_true", help="warm-up and timed steps only (for profiler runs)")
    ap.add_argument("--sweep", default=None, choices=["grid", "configs", "shards", "decode", "bwd"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16", "fp8"], help="--sweep grid")
    ap.add_argument("--gqa", type=int, default=0, help="--sweep grid: number of K/V heads (0: same as query heads)")
    ap.add_argument("--iters", type=int, default=15, help="--sweep: timed launches per cell")
    ap.add_argument("--seq", type=int, default=0, help="--sweep: only this sequence length")
    ap.add_argument("--shards", type=int, default=8, help="--sweep shards: number of K/V shards")
    ap.add_argument("--graph", action="store_true", help="--sweep decode: also time CUDA-graph replays")
    args = ap.parse_args(argv)
    cfg = inputs.CONFIGS[args.config]
    if args.sweep:
        return run_sweep(args)
    if args.impl == "reference":
        return run_reference(args, cfg)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus, argv)
    try:
        return run_stub(args) if args.impl == "stub" else run_ours(args, cfg)
    finally:
        if torch.distributed.is_available() and torch.distributed.is_initialized():
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    sys.exit(main())
