#!/usr/bin/env python
"""Benchmark of the ToMA block path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload cfg3]
    python bench.py --stage attention --workload cfg3 [--full-length] [--ratio 0.25] [--reps 50]   # one stage, one JSON line

A "step" is one toma_block call (Algorithm 3 with the reuse schedule of Sec. 4.3.2)
on one batch of synthetic SDXL-shaped tokens.  Step t of the timed region uses
schedule position t mod 10 of the workload's 10-step sequence, so with reuse
interval 5 two steps in ten recompute selection and weights.  Prints ONE JSON line.

--stage times a single entry point (select, weights, merge, attention, unmerge, block, refresh, linear) with CUDA
events and an L2 flush between repetitions; it is also the small command the ncu captures under profiles/ run.
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
L2_BYTES = 126 << 20   # B200 L2 capacity: independent inputs must exceed it together to count as evicted


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tf_burst": p["bf16_tflops"], "tf_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


def load_traffic():
    """Per-launch DRAM traffic of the dominant kernel, per workload, with the commit and the ncu summary each
    figure comes from (profiles/attention_traffic.json): a figure that has gone stale shows by its source."""
    path = os.path.join(ROOT, "profiles", "attention_traffic.json")
    if os.path.exists(path):
        return json.load(open(path))
    return {}


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


class Timer:
    """CUDA-event timing of a callable on torch's current stream, the L2 flushed (a 256 MB write) before every
    repetition.  The flush also gives the host time to enqueue the call, so the interval is device time."""

    def __init__(self, torch, flush=True):
        self.torch = torch
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda") if flush else None

    def us(self, fn, reps=8, warmup=3):
        """All repetitions' microseconds."""
        torch = self.torch
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        out = []
        for _ in range(reps):
            if self.flush is not None:
                self.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            out.append(1e3 * e0.elapsed_time(e1))
        return out

    def median_us(self, fn, reps=8, warmup=3):
        return statistics.median(self.us(fn, reps, warmup))


def library_attention_us(torch, timer, B, L, heads, dh, x):
    """torch's scaled_dot_product_attention (a library kernel, whichever backend torch picks) on the same
    [B][L][heads][dh] bf16 tensor as Q = K = V: stated context for the full-token comparator, timed outside every
    timed region of the benchmark.  None when torch has no kernel for the shape."""
    try:
        import torch.nn.functional as F
        q = x.view(B, L, heads, dh).permute(0, 2, 1, 3)
        return timer.median_us(lambda: F.scaled_dot_product_attention(q, q, q), reps=8)
    except Exception:
        return None


class Workload:
    """Device tensors of one configuration and the five calls toma_block makes, one by one."""

    def __init__(self, toma, torch, cfg, global_merge=False, weight_reuse_interval=0, x_host=None):
        import gen
        self.toma, self.cfg = toma, cfg
        self.desc = toma.desc_from_config(cfg, weight_reuse_interval=weight_reuse_interval, global_merge=global_merge)
        self.tdt = toma.torch_dtype(self.desc)
        self.x = torch.from_numpy(gen.features(cfg) if x_host is None else x_host).cuda().to(self.tdt)
        self.out = torch.empty_like(self.x)
        self.idx, self.w, self.ws = toma.alloc_idx(self.desc), toma.alloc_weights(self.desc), toma.alloc_workspace(self.desc)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.B, self.N, self.d = cfg.batch, cfg.n_tokens + cfg.n_extra, cfg.dim
        self.d_loc = toma.toma_dest_per_tile(self.desc)
        self.Lm = cfg.n_tiles * self.d_loc + cfg.n_extra
        self.xm = torch.empty((self.B, self.Lm, self.d), dtype=self.tdt, device="cuda")
        self.att = torch.empty_like(self.xm)
        self.o_full = torch.empty_like(self.x)

    def prime(self):
        self.select()
        self.weights()
        self.merge()
        self.attention()

    def select(self):
        self.toma.toma_select(self.desc, self.x, self.idx, self.ws, self.status)

    def weights(self):
        self.toma.toma_merge_weights(self.desc, self.x, self.idx, self.w, self.ws, self.status)

    def merge(self):
        self.toma.toma_merge(self.desc, self.w, self.x, self.xm, self.status)

    def attention(self):
        c = self.cfg
        self.toma.toma_attention(self.B, self.Lm, c.n_heads, c.head_dim, c.dtype, self.xm, self.xm, self.xm, self.att, self.status)

    def full_attention(self):
        c = self.cfg
        self.toma.toma_attention(self.B, self.N, c.n_heads, c.head_dim, c.dtype, self.x, self.x, self.x, self.o_full, self.status)

    def unmerge(self):
        self.toma.toma_unmerge(self.desc, self.w, self.att, self.out, self.status)

    def block(self, step):
        self.toma.toma_block(self.desc, step, self.x, self.out, self.idx, self.w, self.ws, self.status)

    # algorithmic bytes / flops per launch
    def esz(self):
        return 2 if self.cfg.dtype == "bf16" else 4

    def attention_flops(self, L=None):
        L = self.Lm if L is None else L
        return 4.0 * self.B * L * L * self.d

    def merge_bytes(self):   # tokens in, merged tokens out (or the reverse), both weight planes
        c = self.cfg
        return self.B * (c.n_tokens * self.d * self.esz() + c.n_tiles * self.d_loc * self.d * self.esz()
                         + c.n_tiles * c.n_loc * self.d_loc * 4)

    def select_bytes(self):  # tokens in, quantised tokens out and in, similarities out and in, indices out
        c = self.cfg
        return self.B * (c.n_tokens * self.d * (self.esz() + 4) + c.n_tiles * c.n_loc * c.n_loc * 4 + c.n_tiles * self.d_loc * 4)

    def weights_bytes(self):  # tokens in (destinations gathered from them), both weight planes out
        c = self.cfg
        return self.B * (c.n_tokens * self.d * self.esz() + c.n_tiles * self.d_loc * self.d * self.esz()
                         + c.n_tiles * c.n_loc * self.d_loc * 4)


def rooflines(wl, stage_us, peaks):
    """One entry per stage of the path: achieved rate against the measured peak that bounds it."""
    c = wl.cfg
    out = []
    tf = wl.attention_flops() / stage_us["attention"] / 1e6
    out.append({"kernel": "attention_tc_kernel (attention over the merged tokens)", "bound": "tensor", "achieved": tf,
                "peak": peaks["tf_burst"], "unit": "TFLOP/s", "frac": tf / peaks["tf_burst"],
                "frac_of_sustained": tf / peaks["tf_sustained"], "us": stage_us["attention"]})
    for name, nbytes in (("merge", wl.merge_bytes()), ("unmerge", wl.merge_bytes()), ("weights", wl.weights_bytes())):
        gbs = nbytes / stage_us[name] / 1e3
        out.append({"kernel": "toma_" + (name if name != "weights" else "merge_weights"), "bound": "hbm", "achieved": gbs,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": nbytes,
                    "us": stage_us[name]})
    gbs = wl.select_bytes() / stage_us["select"] / 1e3
    out.append({"kernel": "toma_select (quantise + Gram + greedy)", "bound": "latency", "achieved": gbs, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": wl.select_bytes(), "us": stage_us["select"],
                "greedy_rounds": wl.d_loc, "rounds_per_us": wl.d_loc / stage_us["select"],
                "sms_occupied_by_greedy": min(wl.B * c.n_tiles, 148),
                "note": "the greedy loop is sequential in its D_loc rounds: one CTA per tile, bound by the round latency"})
    return out


def attention_back_to_back_us(wl, torch, reps=3):
    """Average duration of the attention launch inside a train of launches: as many independent copies of the
    merged tokens (and outputs) as exceed 1.5 x L2 together take turns, so every launch still finds its operands
    evicted, and ONE event pair brackets the whole train: no per-launch event cost, no exposed launch latency.
    The isolated call of stage_times() is the conservative figure; this one is what the kernel costs in a stream."""
    per = 2 * wl.xm.numel() * wl.xm.element_size()
    n = max(4, -(-int(1.5 * L2_BYTES) // per))
    sets = [(torch.randn_like(wl.xm, dtype=torch.float32).to(wl.xm.dtype), torch.empty_like(wl.xm)) for _ in range(n)]
    c = wl.cfg

    def train():
        for q, o in sets:
            wl.toma.toma_attention(wl.B, wl.Lm, c.n_heads, c.head_dim, c.dtype, q, q, q, o, wl.status)

    train()
    torch.cuda.synchronize()
    best = None
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        train()
        e1.record()
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / n
        best = us if best is None else min(best, us)
    return best, n


def stage_times(wl, timer, reps):
    """Median microseconds of the five calls toma_block makes, each timed alone between L2 flushes."""
    wl.prime()
    return {name: timer.median_us(getattr(wl, name), reps=reps) for name in ("select", "weights", "merge", "attention", "unmerge")}


def block_workload(toma, torch, timer, name, over, reuse, w_reuse, global_merge=False):
    """Block latency vs full-token attention on one configuration (one fixed input; refresh, weights-only and
    reuse steps timed separately, CUDA events, L2 flushed)."""
    import gen
    cfg = gen.config(name, reuse_interval=reuse, **over)
    wl = Workload(toma, torch, cfg, global_merge=global_merge, weight_reuse_interval=w_reuse)
    refresh = timer.median_us(lambda: wl.block(0))
    reuse_us = timer.median_us(lambda: wl.block(1)) if reuse > 1 else None
    n_w = reuse // w_reuse - 1 if w_reuse else 0   # steps that recompute the weights from the cached destinations
    weights_us = timer.median_us(lambda: wl.block(w_reuse)) if n_w else None
    full = timer.median_us(wl.full_attention)
    lib = library_attention_us(torch, timer, wl.B, wl.N, cfg.n_heads, cfg.head_dim, wl.x) if cfg.dtype == "bf16" else None
    mean = refresh if reuse == 1 else (refresh + n_w * (weights_us or 0.0) + (reuse - 1 - n_w) * reuse_us) / reuse
    res = {"tokens": wl.B * wl.N, "tile": [cfg.tile_h, cfg.tile_w], "merge_ratio": cfg.merge_ratio, "global_merge": bool(global_merge),
           "reuse_interval": reuse, "weight_reuse_interval": w_reuse or reuse, "refresh_us": refresh,
           "weights_only_us": weights_us, "reuse_us": reuse_us, "block_mean_us": mean, "full_attention_us": full,
           "full_attention_library_us": lib, "speedup_vs_full_attention": full / mean,
           "speedup_vs_library_full_attention": (lib / mean) if lib else None,
           "tokens_per_s": wl.B * wl.N / (mean * 1e-6), "full_attention_tflops": wl.attention_flops(wl.N) / full / 1e6}
    assert int(wl.status.item()) == 0
    return res, wl


def other_workloads(toma, torch, timer, peaks):
    out = {}
    # cfg2 states no schedule: the paper's weight interval (5) is used.  cfg4 (Flux) does not reuse across
    # timesteps but shares one selection among the blocks of a kind within a step (19 joint blocks).
    # cfg3_stripes: the same tokens cut into stripes of 4 full rows (256 tokens per region, as a 16x16 tile) under
    # the paper's own schedule, destinations every 10 steps and weights every 5.  cfg3_global_merge: the paper's
    # default variant (destinations per 16x16 tile, one dense 2048 x 4096 weight matrix per image), same schedule.
    plans = (("cfg2", "cfg2", {}, 5, 0, False), ("cfg4", "cfg4", {}, 19, 0, False), ("cfg5a", "cfg5a", {}, 5, 0, False),
             ("cfg5b", "cfg5b", {}, 5, 0, False),
             ("cfg3_ratio_0.25", "cfg3", dict(merge_ratio=0.25), 5, 0, False),
             ("cfg3_ratio_0.75", "cfg3", dict(merge_ratio=0.75), 5, 0, False),
             ("cfg3_stripes", "cfg3", dict(tile_h=4, tile_w=64), 10, 5, False),
             ("cfg3_global_merge", "cfg3", {}, 10, 5, True))
    for label, name, over, reuse, w_reuse, gm in plans:
        res, wl = block_workload(toma, torch, timer, name, over, reuse, w_reuse, gm)
        if label in ("cfg4", "cfg5a", "cfg5b"):   # the kernels' rates at the larger sizes
            st = stage_times(wl, timer, reps=5)
            res["stage_us"] = st
            res["rooflines"] = rooflines(wl, st, peaks)
        out[label] = res
        del wl
        torch.cuda.empty_cache()
    out["cfg3_attention_module"] = attention_module_workload(toma, torch, timer)
    out["cfg3_mlp_module"] = mlp_module_workload(toma, torch, timer)
    return out


def attention_module_workload(toma, torch, timer):
    """The benchmark workload with the whole attention module as the wrapped F: Q/K/V projections, attention and
    output projection on the merged tokens (toma_block_proj) against the same module on all tokens
    (toma_attention_proj).  Random N(0, 1/d) projection weights."""
    import gen
    cfg = gen.config("cfg3")
    wl = Workload(toma, torch, cfg)
    d, tdt = cfg.dim, wl.tdt
    ws_w = [torch.from_numpy((gen.normal(0, (96, i, d), d * d).reshape(d, d) / d ** 0.5).astype("float32")).cuda().to(tdt)
            for i in range(4)]
    B, N = cfg.batch, cfg.n_tokens
    ws_full = torch.empty(toma.toma_attention_proj_workspace_bytes(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype),
                          dtype=torch.uint8, device="cuda")
    k = cfg.reuse_interval
    refresh = timer.median_us(lambda: toma.toma_block_proj(wl.desc, 0, wl.x, *ws_w, wl.out, wl.idx, wl.w, wl.ws, None), reps=10)
    reuse_us = timer.median_us(lambda: toma.toma_block_proj(wl.desc, 1, wl.x, *ws_w, wl.out, wl.idx, wl.w, wl.ws, None), reps=10)
    full = timer.median_us(lambda: toma.toma_attention_proj(B, N, cfg.n_heads, cfg.head_dim, cfg.dtype, wl.x, *ws_w, wl.out, ws_full, None), reps=10)
    mean = (refresh + (k - 1) * reuse_us) / k
    m = B * wl.Lm
    qkv = timer.median_us(lambda: toma.toma_linear(wl.x.view(B * N, d)[:m], ws_w[0], wl.out.view(B * N, d)[:m]), reps=10)
    return {"tokens": B * N, "reuse_interval": k, "refresh_us": refresh, "reuse_us": reuse_us, "block_mean_us": mean,
            "full_module_us": full, "speedup_vs_full_module": full / mean,
            "one_projection_us": qkv, "one_projection_tflops": 2.0 * m * d * d / qkv / 1e6}


def mlp_module_workload(toma, torch, timer):
    """The benchmark workload with the MLP as the wrapped F (hidden width 4 d, GELU): toma_block_mlp on the
    merged tokens against the same MLP on all tokens (toma_mlp).  Random N(0, 1/fan-in) weights."""
    import gen
    cfg = gen.config("cfg3")
    wl = Workload(toma, torch, cfg)
    d, f, tdt = cfg.dim, 4 * cfg.dim, wl.tdt
    w1 = torch.from_numpy((gen.normal(0, (99, 1, d, f), d * f).reshape(d, f) / d ** 0.5).astype("float32")).cuda().to(tdt)
    w2 = torch.from_numpy((gen.normal(0, (99, 2, d, f), d * f).reshape(f, d) / f ** 0.5).astype("float32")).cuda().to(tdt)
    B, N = cfg.batch, cfg.n_tokens
    ws_full = torch.empty(toma.toma_mlp_workspace_bytes(B * N, d, f, cfg.dtype), dtype=torch.uint8, device="cuda")
    k = cfg.reuse_interval
    refresh = timer.median_us(lambda: toma.toma_block_mlp(wl.desc, 0, wl.x, w1, w2, wl.out, wl.idx, wl.w, wl.ws, None), reps=10)
    reuse_us = timer.median_us(lambda: toma.toma_block_mlp(wl.desc, 1, wl.x, w1, w2, wl.out, wl.idx, wl.w, wl.ws, None), reps=10)
    full = timer.median_us(lambda: toma.toma_mlp(B * N, d, f, cfg.dtype, wl.x, w1, w2, wl.out, ws_full, None), reps=10)
    mean = (refresh + (k - 1) * reuse_us) / k
    return {"tokens": B * N, "hidden": f, "reuse_interval": k, "refresh_us": refresh, "reuse_us": reuse_us,
            "block_mean_us": mean, "full_module_us": full, "speedup_vs_full_module": full / mean,
            "full_module_tflops": 4.0 * B * N * d * f / full / 1e6}


def run_stage(args):
    """One entry point timed alone (CUDA events, L2 flushed unless --no-flush); prints one JSON line."""
    import torch
    import __graft_entry__ as entry
    entry.build()
    import gen
    import paper_2509_10918_b200 as toma
    timer = Timer(torch, flush=not args.no_flush)
    if args.stage == "linear":   # projection c = a w, bf16
        m, n, k = (int(v) for v in args.mnk.split(","))
        a = torch.randn(m, k, device="cuda").bfloat16()
        wmat = (torch.randn(k, n, device="cuda") / k ** 0.5).bfloat16()
        c = torch.empty(m, n, device="cuda", dtype=torch.bfloat16)
        ts = timer.us(lambda: toma.toma_linear(a, wmat, c), reps=args.reps, warmup=args.warmup)
        med = statistics.median(ts)
        print(json.dumps({"stage": "linear", "m": m, "n": n, "k": k, "median_us": med, "min_us": min(ts),
                          "tflops_median": 2.0 * m * n * k / med / 1e6}))
        return
    cfg = gen.config(args.workload) if args.ratio is None else gen.config(args.workload, merge_ratio=args.ratio)
    wl = Workload(toma, torch, cfg, global_merge=args.global_merge)
    wl.prime()
    calls = {"select": wl.select, "weights": wl.weights, "merge": wl.merge, "unmerge": wl.unmerge,
             "attention": wl.full_attention if args.full_length else wl.attention, "block": lambda: wl.block(1),
             "refresh": lambda: wl.block(0)}
    ts = timer.us(calls[args.stage], reps=args.reps, warmup=args.warmup)
    assert int(wl.status.item()) == 0
    med, mn = statistics.median(ts), min(ts)
    res = {"stage": args.stage, "workload": cfg.name + ("+global" if args.global_merge else ""), "ratio": cfg.merge_ratio,
           "median_us": med, "min_us": mn, "reps": args.reps}
    if args.stage == "attention":
        L = wl.N if args.full_length else wl.Lm
        res.update(length=L, tflops_median=wl.attention_flops(L) / med / 1e6, tflops_best=wl.attention_flops(L) / mn / 1e6)
    elif args.stage in ("merge", "unmerge"):
        res.update(algorithmic_bytes=wl.merge_bytes(), gbs_median=wl.merge_bytes() / med / 1e3, gbs_best=wl.merge_bytes() / mn / 1e3)
    elif args.stage == "select":
        res.update(tiles=wl.B * cfg.n_tiles, rounds=wl.d_loc, us_per_round=med / wl.d_loc)
    print(json.dumps(res))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="toma", choices=["toma", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="skip the secondary workloads")
    ap.add_argument("--stage", default=None, choices=["select", "weights", "merge", "attention", "unmerge", "block", "refresh", "linear"],
                    help="time one entry point alone and print one JSON line for it")
    ap.add_argument("--ratio", type=float, default=None, help="--stage: merge ratio override")
    ap.add_argument("--full-length", action="store_true", help="--stage attention: all N tokens instead of the merged D")
    ap.add_argument("--global-merge", action="store_true", help="--stage: weights / merge / unmerge over the whole image")
    ap.add_argument("--reps", type=int, default=50)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--mnk", default="4096,1920,640", help="--stage linear: rows, columns, contraction length")
    args = ap.parse_args()
    if args.stage:
        run_stage(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "toma" else args.warmup

    import gen
    cfg = gen.config(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

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
    xs_np = list(gen.feature_sequence(cfg_rank, cycle))
    xs_host = [torch.from_numpy(x).to(tdt).pin_memory() for x in xs_np]
    xs = [x.cuda() for x in xs_host]
    out = torch.empty_like(xs[0])
    out_host = torch.empty_like(xs_host[0]).pin_memory()
    idx = toma.alloc_idx(desc)
    w = toma.alloc_weights(desc)
    ws = toma.alloc_workspace(desc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    timer = Timer(torch)
    flush = timer.flush
    B, N = cfg.batch, cfg.n_tokens + cfg.n_extra

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

    # ---- the same K steps back to back, no flush: R independent instances of the block (own tokens, output,
    # state and scratch: consecutive layers of a model), together larger than L2, take turns, so that every step
    # still finds its operands evicted.  One event pair around all K steps: consecutive steps overlap through
    # programmatic dependent launch and no per-step event cost is paid.  Reported beside `value`, not as it.
    def nbytes(*ts):
        return sum(t.numel() * t.element_size() for t in ts)

    inst_bytes = nbytes(xs[0], out, idx, w, ws)
    n_inst = max(2, -(-int(1.5 * L2_BYTES) // inst_bytes))
    inst = [(xs[0].clone(), torch.empty_like(out), toma.alloc_idx(desc), toma.alloc_weights(desc), toma.alloc_workspace(desc))
            for _ in range(n_inst)]

    def inst_step(t):
        x_i, out_i, idx_i, w_i, ws_i = inst[t % n_inst]
        toma.toma_block(desc, (t // n_inst) % cycle, x_i, out_i, idx_i, w_i, ws_i, status)

    for t in range(n_inst):   # every instance's step 0 (a refresh) before the clock starts
        inst_step(t)
    sync_all()
    b2b0, b2b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush.zero_()
    b2b0.record()
    k_b2b = n_inst * cycle   # every instance goes through the whole schedule once
    for t in range(k_b2b):
        inst_step(t)
    b2b1.record()
    sync_all()
    b2b_ms = max_over_ranks(b2b0.elapsed_time(b2b1), dist, "cuda")
    back_to_back = {"ms_per_step": b2b_ms / k_b2b, "value": job_throughput(b2b_ms, k_b2b, B * N, world), "unit": UNIT, "steps": k_b2b,
                    "instances": n_inst, "bytes_per_instance": inst_bytes,
                    "note": "K steps inside one event pair, no flush: independent block instances larger than L2 together take turns"}
    assert int(status.item()) == 0
    del inst
    torch.cuda.empty_cache()

    # ---- per-stage pass and full-token comparators (this rank's batch; outside the timed region) -----------
    wl = Workload(toma, torch, cfg_rank, x_host=xs_np[0])
    reps = min(max(args.steps, 8), 20)
    stage_us = stage_times(wl, timer, reps)
    full_us = timer.median_us(wl.full_attention, reps=reps)
    lib_us = library_attention_us(torch, timer, B, N, cfg.n_heads, cfg.head_dim, wl.x) if cfg.dtype == "bf16" else None
    assert int(wl.status.item()) == 0
    rl = rooflines(wl, stage_us, peaks)
    traffic = load_traffic().get(args.workload, {})
    roofline = {"kernel": rl[0]["kernel"], "bound": "tensor", "achieved": rl[0]["achieved"], "peak": peaks["tf_burst"],
                "unit": "TFLOP/s", "frac": rl[0]["frac"], "traffic": traffic.get("dram_bytes_per_launch"),
                "traffic_source": traffic.get("source"),
                "algorithmic_flops_per_launch": wl.attention_flops(),
                "launch_us": stage_us["attention"],
                "peak_source": peaks["source"] + " bf16 burst (cuBLAS GEMM); the kernel is timed alone between L2 flushes",
                "frac_of_sustained_peak": rl[0]["frac_of_sustained"]}
    b2b_us, b2b_n = attention_back_to_back_us(wl, torch)
    roofline["launch_us_in_a_train"] = b2b_us
    roofline["frac_in_a_train"] = wl.attention_flops() / b2b_us / 1e6 / peaks["tf_burst"]
    roofline["train"] = "%d launches on independent inputs (%.0f MB together, > 1.5 x L2) inside one event pair" % (
        b2b_n, b2b_n * 2 * wl.xm.numel() * wl.xm.element_size() / 1e6)

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
        "full_attention_latency_us": full_us,
        "full_attention_library_us": lib_us,
        "speedup_vs_full_attention": full_us / (1e3 * ms_per_step),
        "speedup_vs_library_full_attention": (lib_us / (1e3 * ms_per_step)) if lib_us else None,
        "comparators": "full_attention_latency_us: this library's attention kernel on all N tokens; "
                       "full_attention_library_us: torch scaled_dot_product_attention on the same tensor (library kernel, context)",
        "back_to_back": back_to_back,
        "stage_us": stage_us,
        "roofline": roofline,
        "rooflines": rl,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": xbytes, "d2h_bytes_per_step": xbytes},
        "gpu_launches": int(gpu_launches),
        "clocks": clocks,
        "paper_context": "paper reports -24%/-23% SDXL/Flux generation latency on RTX6000/V100/RTX8000 (other hardware)",
    }
    if rank == 0 and world == 1 and not args.quick:
        result["other_workloads"] = other_workloads(toma, torch, timer, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(cfg)
    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
