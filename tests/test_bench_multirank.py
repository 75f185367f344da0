"""The N > 1 path of bench.py on CPU: two gloo ranks (replicas only, no data-path collective)."""
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
    # every rank reports its own time; the aggregate uses the slowest one
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 3.0 - rank], world, torch.device("cpu"))
    value = bench.aggregate_throughput(1000, ms / 1e3, world)
    dist.barrier()
    out.put((rank, ms, e2e, value))
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, value in res:
        assert ms == 15.0 and e2e == 3.0                    # the slowest rank's times, on both ranks
        assert abs(value - 2 * 1000 / 0.015) < 1e-6         # work of both replicas over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, torch.device("cpu")) == [1.5, 2.5]
    assert bench.aggregate_throughput(10, 2.0, 1) == 5.0


def test_reference_arm_runs_on_rank_zero_only():
    # under torchrun the other ranks exit 0 without work and print nothing
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
