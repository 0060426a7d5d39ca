"""The multi-GPU path of bench.py: N independent replicas, nothing exchanged but the timings.
Two CPU processes on the gloo backend stand in for two GPUs."""

import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [100.0 + 50.0 * rank, 7.0 - rank]          # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, dist, "cpu")
    q.put((rank, got, bench.whole_job_tokens_per_s(2048, world, got[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_slowest_replica_sets_the_time_and_tokens_add_up():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, tps in res:
        assert got == [150.0, 7.0]
        assert abs(tps - 2 * 2048 / 0.150) < 1e-6


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.whole_job_tokens_per_s(100, 1, 1000.0) == 100.0
