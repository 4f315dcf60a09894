"""The N > 1 plumbing of the benchmark on CPU ranks (gloo, world size 2): times are reduced by
maximum over ranks, throughput counts every rank's replica, and only rank 0 reports."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank, 1.0]
    red = bench.max_over_ranks(mine, world, "cpu")
    dist.barrier()
    out[rank] = red
    dist.destroy_process_group()


def test_times_are_max_over_ranks_and_throughput_counts_all_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0, 1.0]
    sys.path.insert(0, str(ROOT))
    import bench
    # 2 ranks x 1000 units x 3 steps in 11 ms (the slower rank's time)
    assert abs(bench.job_throughput(1000, 3, 2, 11.0) - 2 * 1000 * 3 / 0.011) < 1e-6


def test_reference_arm_reports_once_under_two_ranks():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29733", str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=str(ROOT))
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
