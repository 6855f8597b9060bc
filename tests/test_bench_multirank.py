"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, no GPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu", world)       # rank 1 is the slow one
    rate = bench.whole_job_rate(3.0e9, world, ms)
    dist.barrier()
    dist.destroy_process_group()
    with open(f"{out}.{rank}", "w") as fh:
        json.dump({"ms": ms, "rate": rate}, fh)


def test_max_over_ranks_and_whole_job_rate_with_two_gloo_ranks(tmp_path):
    out = str(tmp_path / "r")
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    for rank in range(2):
        r = json.load(open(f"{out}.{rank}"))
        assert r["ms"] == 15.0                       # every rank sees the slowest rank's time
        assert r["rate"] == 2 * 3.0e9 / 15e-3        # replicas add up over that time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, "cpu", 1) == 7.5
    assert bench.whole_job_rate(1e9, 1, 500.0) == 2e9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_must_match_the_launcher():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2"], env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "torchrun" in r.stderr


def test_step_bytes_formula():
    sys.path.insert(0, ROOT)
    import bench
    # K gradients, K local weights read+written, K pre_weights read, w and mom read+written
    assert bench.step_bytes_per_param(8, 4, 0) == 144
    assert bench.step_bytes_per_param(16, 4, 0) == 272
    assert bench.step_bytes_per_param(16, 4, 2) == 336 and bench.step_bytes_per_param(16, 4, 4) == 336
    assert bench.step_bytes_per_param(32, 2, 0) == 32 * 14 + 16
