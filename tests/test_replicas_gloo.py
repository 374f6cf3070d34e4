"""The multi-GPU mode of bench.py is "replicas only": every rank runs the whole workload, the timed region is
bracketed by barriers, the step time is the MAX over ranks and the reported value the SUM of the ranks'
throughputs at that time. This checks that host logic with two gloo ranks on the CPU."""
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

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 10.0 if rank == 0 else 14.0          # rank 1 is slower
    total = bench.max_over_ranks(my_ms, dist, torch.device("cpu"))
    val = bench.aggregate_value(world, 2_000_000_000, total / 5)
    q.put((rank, total, val))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_sum_at_the_slowest_rank_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total, val in res:
        assert total == 14.0
        assert val == pytest.approx(2 * 2_000_000_000 / (14.0 / 5 * 1e-3) / 1e9)
