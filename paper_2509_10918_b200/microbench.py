"""Per-stage micro-benchmarks of the ToMA path (CUDA events, L2 flushed between repetitions).

    python -m paper_2509_10918_b200.microbench --stage attention --workload cfg3 [--full-length] [--reps 50]
    python -m paper_2509_10918_b200.microbench --stage merge --workload cfg2

Stages: select, weights, merge, attention, unmerge, block, linear (--mnk m,n,k).  Prints one JSON line with median / min
microseconds and the derived GB/s or TFLOP/s.  Also the command to run under ncu when a single
kernel is to be profiled on a small case (--reps 3 --no-flush).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--stage", required=True, choices=["select", "weights", "merge", "attention", "unmerge", "block", "linear"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--ratio", type=float, default=None)
    ap.add_argument("--full-length", action="store_true", help="attention over all N tokens instead of the merged D")
    ap.add_argument("--reps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--global-merge", action="store_true", help="weights / merge / unmerge over the whole image")
    ap.add_argument("--mnk", default="4096,1920,640", help="stage linear: rows, columns, contraction length")
    args = ap.parse_args()

    import torch

    import gen
    import paper_2509_10918_b200 as toma

    if args.stage == "linear":  # projection c = a w, bf16
        m, n, k = (int(v) for v in args.mnk.split(","))
        a = torch.randn(m, k, device="cuda").bfloat16()
        wmat = (torch.randn(k, n, device="cuda") / k ** 0.5).bfloat16()
        c = torch.empty(m, n, device="cuda", dtype=torch.bfloat16)
        flush = None if args.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        times = []
        for it in range(args.warmup + args.reps):
            if flush is not None:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            toma.toma_linear(a, wmat, c)
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(1e3 * e0.elapsed_time(e1))
        med = statistics.median(times)
        print(json.dumps({"stage": "linear", "m": m, "n": n, "k": k, "median_us": med, "min_us": min(times),
                          "tflops_median": 2.0 * m * n * k / med / 1e6}))
        return

    cfg = gen.config(args.workload) if args.ratio is None else gen.config(args.workload, merge_ratio=args.ratio)
    desc = toma.desc_from_config(cfg, global_merge=args.global_merge)
    tdt = toma.torch_dtype(desc)
    x = torch.from_numpy(gen.features(cfg)).cuda().to(tdt)
    out = torch.empty_like(x)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B, N, d = cfg.batch, cfg.n_tokens + cfg.n_extra, cfg.dim
    Lm = (cfg.n_tiles * toma.toma_dest_per_tile(desc)) + cfg.n_extra
    xm = torch.empty((B, Lm, d), dtype=tdt, device="cuda")
    att = torch.empty_like(xm)
    toma.toma_select(desc, x, idx, ws, status)
    toma.toma_merge_weights(desc, x, idx, w, ws, status)
    toma.toma_merge(desc, w, x, xm, status)
    L = N if args.full_length else Lm
    qkv = x if args.full_length else xm
    o = torch.empty_like(qkv)
    toma.toma_attention(B, L, cfg.n_heads, cfg.head_dim, cfg.dtype, qkv, qkv, qkv, o, status)

    calls = {
        "select": lambda: toma.toma_select(desc, x, idx, ws, status),
        "weights": lambda: toma.toma_merge_weights(desc, x, idx, w, ws, status),
        "merge": lambda: toma.toma_merge(desc, w, x, xm, status),
        "attention": lambda: toma.toma_attention(B, L, cfg.n_heads, cfg.head_dim, cfg.dtype, qkv, qkv, qkv, o, status),
        "unmerge": lambda: toma.toma_unmerge(desc, w, o if not args.full_length else att, out, status),
        "block": lambda: toma.toma_block(desc, 1, x, out, idx, w, ws, status),
    }
    fn = calls[args.stage]
    flush = None if args.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    times = []
    for _ in range(args.reps):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(1e3 * e0.elapsed_time(e1))
    assert int(status.item()) == 0
    med, mn = statistics.median(times), min(times)
    esz = 2 if cfg.dtype == "bf16" else 4
    res = {"stage": args.stage, "workload": cfg.name + ("+global" if args.global_merge else ""), "ratio": cfg.merge_ratio, "median_us": med, "min_us": mn,
           "reps": args.reps}
    if args.stage == "attention":
        flops = 4.0 * B * L * L * d
        res.update(length=L, tflops_median=flops / med / 1e6, tflops_best=flops / mn / 1e6)
    elif args.stage in ("merge", "unmerge"):
        wbytes = 4 if cfg.dtype == "bf16" else 4
        nbytes = B * (cfg.n_tokens * d * esz + (cfg.n_tiles * toma.toma_dest_per_tile(desc)) * d * esz + cfg.n_tiles * cfg.n_loc * toma.toma_dest_per_tile(desc) * wbytes)
        res.update(algorithmic_bytes=nbytes, gbs_median=nbytes / med / 1e3, gbs_best=nbytes / mn / 1e3)
    elif args.stage == "select":
        res.update(tiles=B * cfg.n_tiles, rounds=toma.toma_dest_per_tile(desc), us_per_round=med / toma.toma_dest_per_tile(desc))
    print(json.dumps(res))


if __name__ == "__main__":
    main()
