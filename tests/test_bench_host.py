"""Host-side logic of the multi-GPU benchmark path, on CPU with gloo and two ranks: every rank
gets its own batch, the job time is the slowest rank's, throughput counts all ranks' tokens."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import gen
    cfg = gen.config("cfg2", grid_h=8, grid_w=8, dim=64, n_heads=1)
    mine = bench.rank_config(cfg, rank)
    x = gen.features(mine)
    local_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
    total = bench.max_over_ranks(local_ms, dist, "cpu")
    value = bench.job_throughput(total, 5, 1000, world)
    gathered = [None] * world
    dist.all_gather_object(gathered, float(np.abs(x).sum()))
    out.put((rank, total, value, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_weak_scaling_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total, value, sums in res:
        assert total == 20.0                           # max over ranks
        assert value == 2 * 1000 * 5 / 0.020           # both ranks' tokens over the slowest time
        assert sums[0] != sums[1]                      # the ranks really hold different batches


def test_reference_arm_non_zero_ranks_do_nothing(monkeypatch, capsys):
    import argparse
    import bench
    import gen
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(argparse.Namespace(steps=1, warmup=0, gpus=2), gen.config("cfg2"))
    assert capsys.readouterr().out == ""


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` (the oracle on the host cores, no GPU involved) prints one JSON line with
    the keys the benchmark contract names."""
    import json
    import subprocess
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "toma_block_tokens_per_s" and line["unit"] == "tokens/s"
    for key in ("value", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype",
                "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["value"] > 0 and line["config"]["workload"].startswith("cfg3")
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
