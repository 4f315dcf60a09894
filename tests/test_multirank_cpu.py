"""The N > 1 plumbing of the benchmark on CPU ranks (gloo, world size 2): times are reduced by
maximum over ranks, throughput counts every rank's replica, only rank 0 reports, and `--gpus N` started
without a launcher becomes N ranks."""
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


def test_gpus_flag_without_launcher_spawns_the_ranks():
    # `python bench.py --gpus 2` with no WORLD_SIZE in the environment: the script re-executes itself under
    # torch.distributed.run with two ranks (CPU ranks here: the reference arm needs no GPU); one line, n_gpus = 2
    sys.path.insert(0, str(ROOT))
    import bench
    cmd = bench.launcher_command(2, ["--gpus", "2", "--steps", "1"], 29741)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "2" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "1"] and cmd[-5].endswith("bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=str(ROOT), env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2


def test_rank_count_must_match_the_gpus_asked_for():
    sys.path.insert(0, str(ROOT))
    import bench
    import pytest
    bench.check_world(1, 1)
    bench.check_world(4, 4)
    with pytest.raises(SystemExit):
        bench.check_world(8, 1)          # asked for 8 GPUs, one rank running: never reported as n_gpus = 1


def test_both_arms_print_one_config(tmp_path):
    # the CUDA arm and the reference arm describe the workload with one function: same keys, same values
    sys.path.insert(0, str(ROOT))
    import bench
    from paper_2310_02409_b200 import inputs
    wl = inputs.WORKLOADS[bench.WORKLOAD]
    a = bench.workload_config(wl, 205, 8, 1)
    assert a["workload"] == "c2_llama7b_decode" and a["nuggets_per_seq"] == 205 and a["instances"] == 8
    assert "282 MB" in a["l2"]          # 8 x 2 x 8 x (205 + 64) rows of 8 KB
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600, cwd=str(ROOT))
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][0])
    assert d["config"] == a
