"""Host logic of a multi-replica benchmark run (bench.py --gpus N), on CPU with the gloo backend.

The path has no exchange step: every rank trains its own replica on its own batch.  What the ranks
share is the timing rule: the job's time is the maximum over the ranks, its throughput the units of
all ranks over that time, and rank 0 alone prints.  Two processes stand in for two GPUs."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (r + 1) ms on the device and (10 - r) ms end to end
    dev_ms, e2e_ms = bench.max_over_ranks([rank + 1.0, 10.0 - rank], world, "cpu")
    seed = bench.replica_seed(7, rank)
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{dev_ms} {e2e_ms} {seed} {bench.whole_job_rate(128, world, 5, dev_ms)}")
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_add_their_units(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [open(tmp_path / f"rank{r}.txt").read().split() for r in range(world)]
    for r in range(world):
        assert float(got[r][0]) == 2.0 and float(got[r][1]) == 10.0          # the maximum over both ranks, on every rank
        assert float(got[r][3]) == 128 * 2 * 5 / 2e-3                          # units of both replicas over the slowest time
    assert int(got[0][2]) != int(got[1][2])                                  # different batches per replica


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks([3.5, 1.25], 1, "cpu") == [3.5, 1.25]
    assert bench.whole_job_rate(64, 1, 10, 500.0) == 1280.0


def test_reference_arm_runs_on_rank_zero_only():
    """Under torchrun every rank starts bench.py --impl reference; only rank 0 works and prints."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
