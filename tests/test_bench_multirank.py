"""Host-side logic of bench.py for more than one rank, run as two `gloo` processes on the CPU: the job time is the MAX
over ranks, the aggregate counts every rank's work, and the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]         # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, world, torch.device("cpu"))
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump(got, f)
    dist.barrier()
    dist.destroy_process_group()


def test_job_time_is_the_max_over_ranks(tmp_path):
    world, port = 2, 29541
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        with open(tmp_path / f"rank{rank}.json") as f:
            assert json.load(f) == [15.0, 100.0]


def test_aggregate_counts_every_rank():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.aggregate_value(1e12, steps=10, world=1, total_ms=1000.0)
    two = bench.aggregate_value(1e12, steps=10, world=2, total_ms=1000.0)
    assert one == 10.0 and two == 20.0
    assert bench.max_over_ranks([3.0, 4.0], 1, torch.device("cpu")) == [3.0, 4.0]


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "3"], capture_output=True, text=True, env=env, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
