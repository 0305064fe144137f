"""Throughput sweep over the benchmark grid of the paper's Section 4.1.

    python -m paper_2506_12355_b200.sweep [--dtype bf16|fp16|fp8] [--gqa Hkv] [--iters N] [--seq S] [--shards N] [--decode] [--configs]

Grid: sequence length 512 .. 16k with the batch chosen so that batch x sequence = 16k tokens,
hidden size 2048 (32 heads of dim 64 or 16 heads of dim 128), with and without the causal mask; in
addition head dim 256 (8 heads) and the 192/128 MLA head shape (16 heads); `--dtype fp8` runs the
configuration of the paper's FP8 case study (Section 4.4, Table 6: 16 heads of dim 128) on E4M3
inputs.  FLOPs are counted as in
the paper, 4 * seq^2 * head_dim * heads per batch element, halved for the causal rows (for the
192/128 shape: 2 * seq^2 * (192 + 128) * heads).  Inputs are seeded N(0,1) values; every shape is
timed with CUDA events over isolated launches with a buffer larger than L2 rewritten in between.

`--shards N` times the K/V-sharded path instead (the building block of split-KV decoding and of K/V
sharding across GPUs): N partial launches over N key ranges of one problem (causal, 32 heads of dim
128, bf16) and the merge of their results, against the unsharded call; the merge kernel is
memory-bound and is reported in GB/s of the bytes it must move.

`--configs` times the five benchmark configurations C1..C5 the same way (isolated launches, L2 flushed).

`--decode` times decoding shapes (one query per head, long key/value cache, bf16, head dim 128) through
`attn_fwd_splitkv` for several numbers of key ranges: with one query row per head the work is reading K
and V once, so the figure of merit is GB/s of K and V bytes against the memory bandwidth.
"""
from __future__ import annotations

import argparse

import torch

from . import api, inputs


def time_call(fn, flush, iters):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    ts = []
    for i in range(iters):
        flush.fill_(i & 0xff)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ts.sort()
    return ts[len(ts) // 2]


def shard_table(args, dev, flush):
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

        t_full = time_call(lambda: api.attn_fwd(q, k, v, scale, True, out=o, lse=lse), flush, args.iters)
        t_part = time_call(partials, flush, args.iters)
        t_merge = time_call(lambda: api.attn_combine(o_parts, l_parts, out=o, lse=lse), flush, args.iters)
        moved = (n + 1) * H * S * (D * 2 + 4)
        print("| %d | %.3f | %.3f | %.1f | %.0f | %.2f |" % (S, t_full, t_part, t_merge * 1e3, moved / t_merge / 1e6,
                                                       (t_part + t_merge) / t_full), flush=True)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status")


def decode_table(args, dev, flush):
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
            ms = time_call(lambda: api.attn_fwd_splitkv(q, k, v, D ** -0.5, False, n, workspace=ws, out=o, lse=lse),
                           flush, args.iters)
            cells.append("%.0f (%.0f)" % (ms * 1e3, kv_bytes / ms / 1e6))
        print("| %d x %d (%d) x %d | %.0f | %s |" % (B, H, Hkv, Sk, kv_bytes / 1e6, " | ".join(cells)), flush=True)
        del q, k, v, o, lse, ws
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16", "fp8"])
    ap.add_argument("--gqa", type=int, default=0, help="number of K/V heads (0: same as query heads)")
    ap.add_argument("--iters", type=int, default=15)
    ap.add_argument("--seq", type=int, default=0, help="only this sequence length (a power of two, 512..16384)")
    ap.add_argument("--shards", type=int, default=0, help="time N K/V shards + merge against the unsharded call")
    ap.add_argument("--decode", action="store_true", help="decoding shapes through attn_fwd_splitkv")
    ap.add_argument("--configs", action="store_true", help="the benchmark configurations C1..C5, isolated launches")
    args = ap.parse_args()
    dt = inputs.DTYPE_BF16 if args.dtype == "bf16" else inputs.DTYPE_FP16
    dev = torch.device("cuda:0")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    if args.shards:
        shard_table(args, dev, flush)
        return
    if args.decode:
        decode_table(args, dev, flush)
        return
    if args.configs:
        print("| config | time | TFLOP/s | GB/s at algorithmic bytes |")
        print("|---|---|---|---|")
        for name in sorted(inputs.CONFIGS):
            cfg = inputs.CONFIGS[name]
            q, k, v = (t.to(dev) for t in inputs.make_config_inputs(cfg))
            o = torch.empty_like(q)
            lse = torch.empty((cfg.B, cfg.H, cfg.Sq), dtype=torch.float32, device=dev)
            ms = time_call(lambda: api.attn_fwd(q, k, v, cfg.scale, cfg.causal, out=o, lse=lse), flush, max(args.iters, 30))
            print("| %s | %.1f us | %.1f | %.0f |" % (cfg.workload, ms * 1e3, cfg.flops / ms / 1e9, cfg.min_hbm_bytes / ms / 1e6), flush=True)
            del q, k, v, o, lse
        if api.attn_last_device_status() != 0:
            raise SystemExit("device timeout status")
        return
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
                    fn = lambda: api.attn_fwd_fp8(q, k, v, scale, 1.0, 1.0, 1.0, causal, out=o, lse=lse)
                elif Dqk == Dv:
                    fn = lambda: api.attn_fwd_gqa(q, k, v, scale, causal, out=o, lse=lse)
                else:
                    fn = lambda: api.attn_fwd_qkv_dims(q, k, v, scale, causal, out=o, lse=lse)
                ms = time_call(fn, flush, args.iters)
                flops = 2.0 * B * H * S * S * (Dqk + Dv) / (2 if causal else 1)
                cells.append("%.0f" % (flops / ms / 1e9))
                del q, k, v, o, lse
            print("| %d x %s%s | %s | %s |" % (H, name, "" if Hkv == H else " (Hkv=%d)" % Hkv,
                                              "causal" if causal else "none", " | ".join(cells)), flush=True)
    if api.attn_last_device_status() != 0:
        raise SystemExit("device timeout status")


if __name__ == "__main__":
    main()
