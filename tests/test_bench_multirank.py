"""CPU test of the N > 1 path of bench.py: ranks are independent replicas, the reported time is
the maximum over ranks and the value is the aggregate over all ranks (world size 2, gloo)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per_rank_us = 100.0 + 50.0 * rank          # rank 1 is the slow replica
    slowest = bench.max_over_ranks(per_rank_us, dist, "cpu")
    dist.barrier()
    q.put((rank, slowest, bench.whole_job_tflops(world, 2.0e12, slowest * 1e-6)))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 150.0                               # max over ranks, on every rank
        assert value == pytest.approx(2 * 2.0e12 / 150e-6 / 1e12)


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_tflops(1, 34.36e9, 57.3e-6) == pytest.approx(599.65, rel=1e-3)
    rank, local, world = bench._dist_env()
    assert world >= 1
