"""Host logic of the multi-rank benchmark path, on CPU with the gloo backend (world size 2):
replicas share nothing, the job's time is the slowest rank's and its tokens are the sum."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, value = bench.aggregate_replicas([10.0, 30.0][rank], [600, 500][rank], world, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "value": value}, f)


def test_two_ranks_take_max_time_and_sum_tokens(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        got = json.load(open(tmp_path / f"r{r}.json"))
        assert got["ms"] == 30.0
        assert abs(got["value"] - 1100 / 0.030) < 1e-6


def test_single_rank_is_untouched():
    import bench
    ms, value = bench.aggregate_replicas(20.0, 100, 1, torch.device("cpu"))
    assert ms == 20.0 and abs(value - 5000.0) < 1e-9


def test_reference_arm_only_runs_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
