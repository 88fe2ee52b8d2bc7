#!/usr/bin/env python
"""Benchmark of the ToMA block path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload cfg3]

A "step" is one toma_block call (Algorithm 3 with the reuse schedule of Sec. 4.3.2)
on one batch of synthetic SDXL-shaped tokens.  Step t of the timed region uses
schedule position t mod 10 of the workload's 10-step sequence, so with reuse
interval 5 two steps in ten recompute selection and weights.  Prints ONE JSON line.
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

METRIC = "toma_block_tokens_per_s"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tf_burst": p["bf16_tflops"], "tf_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_step_seconds(cfg, x_host, step, state):
    from oracle import toma_oracle as O
    t0 = time.perf_counter()
    O.block_step(x_host, step, state, grid_h=cfg.grid_h, grid_w=cfg.grid_w, tile_h=cfg.tile_h, tile_w=cfg.tile_w,
                 merge_ratio=cfg.merge_ratio, tau=cfg.tau, n_heads=cfg.n_heads, reuse_interval=cfg.reuse_interval,
                 n_extra=cfg.n_extra)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(cfg):
    """The oracle as it stands, timed on this machine's host cores over the workload's whole step schedule
    (two refresh and eight reuse steps of the full batch: about ten seconds of CPU work)."""
    import gen
    from oracle import toma_oracle as O
    seq = list(gen.feature_sequence(cfg, cfg.steps))
    st = O.BlockState()
    times = [oracle_step_seconds(cfg, x, t, st) for t, x in enumerate(seq)]
    k = cfg.reuse_interval
    refresh = [dt for t, dt in enumerate(times) if t % k == 0]
    reuse = [dt for t, dt in enumerate(times) if t % k != 0]
    tokens = len(seq) * cfg.batch * (cfg.n_tokens + cfg.n_extra)
    t_refresh = sum(refresh) / max(len(refresh), 1)
    t_reuse = sum(reuse) / max(len(reuse), 1)
    return {"value": tokens / sum(times), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"the whole schedule once, all {cfg.batch} batch items: {len(refresh)} refresh steps ({t_refresh:.2f} s each) "
                      f"and {len(reuse)} reuse steps ({t_reuse:.2f} s each), {sum(times):.1f} s in all",
            "refresh_s": t_refresh, "reuse_s": t_reuse}


def run_reference(args, cfg):
    """The CPU oracle as the reference arm: each step is schedule step t on batch item 0."""
    import gen
    from oracle import toma_oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    seq = list(gen.feature_sequence(cfg, cfg.steps))
    st = O.BlockState()
    cycle = cfg.steps
    for t in range(args.warmup):
        oracle_step_seconds(cfg, seq[t % cycle][:1], t % cycle, st)
    t0 = time.perf_counter()
    for t in range(args.steps):
        oracle_step_seconds(cfg, seq[t % cycle][:1], t % cycle, st)
    dt = time.perf_counter() - t0
    tokens = cfg.n_tokens + cfg.n_extra
    value = tokens * args.steps / dt
    sample = f"batch item 0 of {cfg.batch} per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def rank_config(cfg, rank: int):
    """Weak scaling: every rank works on its own batch of the same shape (its own random stream)."""
    return cfg.with_(seed=cfg.seed + rank)


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's time (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(total_ms: float, steps: int, tokens_per_rank_step: int, world: int) -> float:
    """Whole-job tokens/s: all ranks' tokens over the slowest rank's time."""
    return world * tokens_per_rank_step * steps / (total_ms * 1e-3)


def workload_config(cfg):
    return {"workload": f"{cfg.name}: SDXL-like high-resolution block, batch {cfg.batch}, {cfg.grid_h}x{cfg.grid_w} "
                        f"tokens, d={cfg.dim} {cfg.dtype}, {cfg.n_heads}x{cfg.head_dim} heads, tiles "
                        f"{cfg.tile_h}x{cfg.tile_w}, merge ratio {cfg.merge_ratio}, reuse interval "
                        f"{cfg.reuse_interval} over a {cfg.steps}-step drifting sequence",
            "global_batch": cfg.batch, "seq_len": cfg.n_tokens + cfg.n_extra, "l2": "flushed between steps",
            "parallelism": "independent batches per GPU, no collective"}


def other_workloads(toma, torch, flush, peaks):
    """Block latency vs full-token attention on the other SDXL- and Flux-shaped configurations
    (one fixed input per workload; refresh and reuse steps timed separately, CUDA events, L2 flushed)."""
    import gen
    out = {}
    # cfg2 states no schedule: the paper's weight interval (5) is used.  cfg4 (Flux) does not reuse across
    # timesteps but shares one selection among the blocks of a kind within a step (19 joint blocks).
    # cfg3_stripes: the same tokens cut into stripes of 4 full rows (256 tokens per region, as a 16x16 tile) under
    # the paper's own schedule, destinations every 10 steps and weights every 5.  cfg3_global_merge: the paper's
    # default variant (destinations per 16x16 tile, one dense 2048 x 4096 weight matrix per image), same schedule.
    for label, name, over, reuse, w_reuse in (("cfg2", "cfg2", {}, 5, 0), ("cfg4", "cfg4", {}, 19, 0),
                                              ("cfg5a", "cfg5a", {}, 5, 0),
                                              ("cfg3_stripes", "cfg3", dict(tile_h=4, tile_w=64), 10, 5),
                                              ("cfg3_global_merge", "cfg3", dict(global_merge=True), 10, 5)):
        global_merge = over.pop("global_merge", False) if isinstance(over, dict) else False
        cfg = gen.config(name, reuse_interval=reuse, **over)
        desc = toma.desc_from_config(cfg, weight_reuse_interval=w_reuse, global_merge=global_merge)
        tdt = toma.torch_dtype(desc)
        x = torch.from_numpy(gen.features(cfg)).cuda().to(tdt)
        y = torch.empty_like(x)
        idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
        B, N, d = cfg.batch, cfg.n_tokens + cfg.n_extra, cfg.dim

        def t_us(fn, reps=8):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            ts = []
            for _ in range(reps):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                ts.append(1e3 * e0.elapsed_time(e1))
            return statistics.median(ts)

        refresh = t_us(lambda: toma.toma_block(desc, 0, x, y, idx, w, ws, None))
        reuse_us = t_us(lambda: toma.toma_block(desc, 1, x, y, idx, w, ws, None)) if reuse > 1 else None
        # steps that recompute the weights from the cached destinations
        n_w = reuse // w_reuse - 1 if w_reuse else 0
        weights_us = t_us(lambda: toma.toma_block(desc, w_reuse, x, y, idx, w, ws, None)) if n_w else None
        full = t_us(lambda: toma.toma_attention(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype, x, x, x, y, None))
        mean = refresh if reuse == 1 else (refresh + n_w * (weights_us or 0.0) + (reuse - 1 - n_w) * reuse_us) / reuse
        out[label] = {"tokens": B * N, "tile": [cfg.tile_h, cfg.tile_w], "global_merge": bool(global_merge),
                      "reuse_interval": reuse,
                      "weight_reuse_interval": w_reuse or reuse, "refresh_us": refresh, "weights_only_us": weights_us,
                      "reuse_us": reuse_us, "block_mean_us": mean, "full_attention_us": full,
                      "speedup_vs_full_attention": full / mean, "tokens_per_s": B * N / (mean * 1e-6),
                      "full_attention_tflops": 4.0 * B * N * N * d / full / 1e6}
        del x, y, idx, w, ws
        torch.cuda.empty_cache()
    out["cfg3_attention_module"] = attention_module_workload(toma, torch, flush)
    out["cfg3_mlp_module"] = mlp_module_workload(toma, torch, flush)
    return out


def attention_module_workload(toma, torch, flush):
    """The benchmark workload with the whole attention module as the wrapped F: Q/K/V projections, attention and
    output projection on the merged tokens (toma_block_proj) against the same module on all tokens
    (toma_attention_proj).  Random N(0, 1/d) projection weights."""
    import gen
    cfg = gen.config("cfg3")
    desc = toma.desc_from_config(cfg)
    tdt = toma.torch_dtype(desc)
    x = torch.from_numpy(gen.features(cfg)).cuda().to(tdt)
    y = torch.empty_like(x)
    d = cfg.dim
    ws_w = [torch.from_numpy((gen.normal(0, (96, i, d), d * d).reshape(d, d) / d ** 0.5).astype("float32")).cuda().to(tdt)
            for i in range(4)]
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    B, N = cfg.batch, cfg.n_tokens
    ws_full = torch.empty(toma.toma_attention_proj_workspace_bytes(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype),
                          dtype=torch.uint8, device="cuda")

    def t_us(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        return statistics.median(ts)

    k = cfg.reuse_interval
    refresh = t_us(lambda: toma.toma_block_proj(desc, 0, x, *ws_w, y, idx, w, ws, None))
    reuse_us = t_us(lambda: toma.toma_block_proj(desc, 1, x, *ws_w, y, idx, w, ws, None))
    full = t_us(lambda: toma.toma_attention_proj(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype, x, *ws_w, y, ws_full, None))
    mean = (refresh + (k - 1) * reuse_us) / k
    m = B * (cfg.n_tiles * toma.toma_dest_per_tile(desc) + cfg.n_extra)
    qkv = t_us(lambda: toma.toma_linear(x.view(B * N, d)[:m], ws_w[0], y.view(B * N, d)[:m]))
    return {"tokens": B * N, "reuse_interval": k, "refresh_us": refresh, "reuse_us": reuse_us, "block_mean_us": mean,
            "full_module_us": full, "speedup_vs_full_module": full / mean,
            "one_projection_us": qkv, "one_projection_tflops": 2.0 * m * d * d / qkv / 1e6}


def mlp_module_workload(toma, torch, flush):
    """The benchmark workload with the MLP as the wrapped F (hidden width 4 d, GELU): toma_block_mlp on the
    merged tokens against the same MLP on all tokens (toma_mlp).  Random N(0, 1/fan-in) weights."""
    import gen
    cfg = gen.config("cfg3")
    desc = toma.desc_from_config(cfg)
    tdt = toma.torch_dtype(desc)
    x = torch.from_numpy(gen.features(cfg)).cuda().to(tdt)
    y = torch.empty_like(x)
    d, f = cfg.dim, 4 * cfg.dim
    w1 = torch.from_numpy((gen.normal(0, (99, 1, d, f), d * f).reshape(d, f) / d ** 0.5).astype("float32")).cuda().to(tdt)
    w2 = torch.from_numpy((gen.normal(0, (99, 2, d, f), d * f).reshape(f, d) / f ** 0.5).astype("float32")).cuda().to(tdt)
    idx, w, ws = toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc)
    B, N = cfg.batch, cfg.n_tokens
    ws_full = torch.empty(toma.toma_mlp_workspace_bytes(B * N, d, f, cfg.dtype), dtype=torch.uint8, device="cuda")

    def t_us(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(1e3 * e0.elapsed_time(e1))
        return statistics.median(ts)

    k = cfg.reuse_interval
    refresh = t_us(lambda: toma.toma_block_mlp(desc, 0, x, w1, w2, y, idx, w, ws, None))
    reuse_us = t_us(lambda: toma.toma_block_mlp(desc, 1, x, w1, w2, y, idx, w, ws, None))
    full = t_us(lambda: toma.toma_mlp(B * N, d, f, cfg.dtype, x, w1, w2, y, ws_full, None))
    mean = (refresh + (k - 1) * reuse_us) / k
    return {"tokens": B * N, "hidden": f, "reuse_interval": k, "refresh_us": refresh, "reuse_us": reuse_us,
            "block_mean_us": mean, "full_module_us": full, "speedup_vs_full_module": full / mean,
            "full_module_tflops": 4.0 * B * N * d * f / full / 1e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="toma", choices=["toma", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="skip the secondary workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "toma" else args.warmup

    import gen
    cfg = gen.config(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import numpy as np
    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2509_10918_b200 as toma

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the ToMA path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    peaks = load_peaks()
    cfg_rank = rank_config(cfg, rank)
    desc = toma.desc_from_config(cfg_rank)
    tdt = toma.torch_dtype(desc)
    cycle = cfg.steps
    xs_host = [torch.from_numpy(x).to(tdt).pin_memory() for x in gen.feature_sequence(cfg_rank, cycle)]
    xs = [x.cuda() for x in xs_host]
    out = torch.empty_like(xs[0])
    out_host = torch.empty_like(xs_host[0]).pin_memory()
    idx = toma.alloc_idx(desc)
    w = toma.alloc_weights(desc)
    ws = toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    B, N, d = cfg.batch, cfg.n_tokens + cfg.n_extra, cfg.dim
    d_loc = toma.toma_dest_per_tile(desc)
    Lm = cfg.n_tiles * d_loc + cfg.n_extra

    def block(t):
        toma.toma_block(desc, t % cycle, xs[t % cycle], out, idx, w, ws, status)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for t in range(warmup):
            fn(t)
        sync_all()
        evs = []
        for t in range(steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(t)
            e1.record()
            evs.append((e0, e1))
        sync_all()
        return [a.elapsed_time(b) for a, b in evs]

    # ---- the timed region: K toma_block steps -------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = toma.toma_launch_counter()
    for t in range(args.warmup):
        block(t)
    launches_warm = toma.toma_launch_counter() - launches0
    step_ms = timed(block, args.steps, 0)
    gpu_launches = toma.toma_launch_counter() - launches0 - launches_warm
    clocks = sampler.stop()
    assert int(status.item()) == 0, "a kernel reported a device-side timeout"
    total_ms = max_over_ranks(sum(step_ms), dist, "cuda")
    ms_per_step = total_ms / args.steps
    value = job_throughput(total_ms, args.steps, B * N, world)
    refresh_ms = [m for t, m in enumerate(step_ms) if (t % cycle) % cfg.reuse_interval == 0]
    reuse_ms = [m for t, m in enumerate(step_ms) if (t % cycle) % cfg.reuse_interval != 0]

    # ---- full-token attention with the same kernel at length N --------------------------------
    o_full = torch.empty_like(xs[0])

    def full_attention(t):
        x = xs[t % cycle]
        toma.toma_attention(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype, x, x, x, o_full, status)

    full_ms = timed(full_attention, min(args.steps, 20), 3)

    # ---- per-stage breakdown (same calls toma_block makes, events in between) -------------------
    xm = torch.empty((B, Lm, d), dtype=tdt, device="cuda")
    att = torch.empty_like(xm)
    stages = {"select": [], "weights": [], "merge": [], "attention": [], "unmerge": []}
    reps = min(args.steps, 20)
    for t in range(3 + reps):
        x = xs[t % cycle]
        flush.zero_()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        ev[0].record()
        toma.toma_select(desc, x, idx, ws, status)
        ev[1].record()
        toma.toma_merge_weights(desc, x, idx, w, ws, status)
        ev[2].record()
        toma.toma_merge(desc, w, x, xm, status)
        ev[3].record()
        toma.toma_attention(B, Lm, cfg.n_heads, cfg.head_dim, cfg.dtype, xm, xm, xm, att, status)
        ev[4].record()
        toma.toma_unmerge(desc, w, att, out, status)
        ev[5].record()
        torch.cuda.synchronize()
        if t >= 3:
            for i, name in enumerate(stages):
                stages[name].append(ev[i].elapsed_time(ev[i + 1]))
    stage_ms = {k: statistics.median(v) for k, v in stages.items()}
    esz = 2 if cfg.dtype == "bf16" else 4
    att_flops = 4.0 * B * Lm * Lm * d
    att_tf = att_flops / (stage_ms["attention"] * 1e-3) / 1e12
    mrg_bytes = B * (cfg.n_tokens * d * esz + cfg.n_tiles * d_loc * d * esz + cfg.n_tiles * cfg.n_loc * d_loc * esz)
    # traffic: dram__bytes_read.sum + dram__bytes_write.sum of one launch of this kernel on this workload,
    # from the ncu capture summarised in profiles/attention_tc_cfg3_cfg5a.md (only valid for the default workload)
    traffic = 5331200 + 225024 if args.workload == "cfg3" else None
    roofline = {"kernel": "attention over merged tokens", "bound": "tensor", "achieved": att_tf,
                "peak": peaks["tf_burst"], "unit": "TFLOP/s", "frac": att_tf / peaks["tf_burst"], "traffic": traffic,
                "algorithmic_flops_per_launch": att_flops,
                "peak_source": peaks["source"] + " bf16 burst",
                "merge_gbs": mrg_bytes / (stage_ms["merge"] * 1e-3) / 1e9,
                "unmerge_gbs": mrg_bytes / (stage_ms["unmerge"] * 1e-3) / 1e9,
                "hbm_peak_gbs": peaks["hbm_gbs"]}

    # ---- end to end: pinned host input -> device -> block -> host output, every step ----------
    # One toma_block_host call per step (host pointers through the C ABI).  Copy-in, kernels and copy-out
    # run on three streams chained by the call; two sets of staging buffers let step t+1's copy-in and
    # step t-1's copy-out overlap step t's kernels.  The waits below order the reuse of a staging buffer.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    x_stage = [torch.empty_like(xs[0]) for _ in range(2)]
    out_stage = [torch.empty_like(xs[0]) for _ in range(2)]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    for e in ev_in + ev_done + ev_out:
        e.record()  # creates the handles; everything before the loop is complete by then

    def e2e_step(t):
        k = t % 2
        s_in.wait_event(ev_done[k])                          # kernels of step t-2 have read x_stage[k]
        torch.cuda.current_stream().wait_event(ev_out[k])    # copy-out of step t-2 has read out_stage[k]
        toma.toma_block_host(desc, t % cycle, xs_host[t % cycle], out_host, x_stage[k], out_stage[k], idx, w, ws, status,
                             s_in, s_out, ev_in[k], ev_done[k])
        ev_out[k].record(s_out)

    for t in range(3):
        e2e_step(t)
    sync_all()
    t0 = time.perf_counter()
    for t in range(args.steps):
        e2e_step(t)
    sync_all()
    e2e_s = time.perf_counter() - t0
    e2e_value = job_throughput(1e3 * max_over_ranks(e2e_s, dist, "cuda"), args.steps, B * N, world)
    xbytes = xs[0].numel() * xs[0].element_size()

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic", "config": workload_config(cfg),
        "block_latency_us": {"mean": 1e3 * ms_per_step, "refresh_median": 1e3 * statistics.median(refresh_ms) if refresh_ms else None,
                             "reuse_median": 1e3 * statistics.median(reuse_ms) if reuse_ms else None},
        "full_attention_latency_us": 1e3 * statistics.median(full_ms),
        "speedup_vs_full_attention": statistics.median(full_ms) / ms_per_step,
        "stage_us": {k: 1e3 * v for k, v in stage_ms.items()},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": xbytes, "d2h_bytes_per_step": xbytes},
        "gpu_launches": int(gpu_launches),
        "clocks": clocks,
        "paper_context": "paper reports -24%/-23% SDXL/Flux generation latency on RTX6000/V100/RTX8000 (other hardware)",
    }
    if rank == 0 and world == 1 and not args.quick:
        result["other_workloads"] = other_workloads(toma, torch, flush, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(cfg)
    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
