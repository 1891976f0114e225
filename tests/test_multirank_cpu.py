"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The layer does not shard (one GPU, no collective on the data path), so several GPUs run
independent replicas; what the ranks share is only the timing: a barrier on both sides of the
timed region and the maximum over the ranks' times.  These tests run that logic as two
processes over gloo.
"""
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
    try:
        dist.barrier()
        my_ms = 10.0 + 5.0 * rank                    # rank 1 is the slow replica
        ms = bench.max_over_ranks(my_ms, dist, "cpu")
        dist.barrier()
        q.put((rank, ms, bench.job_throughput(256, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_replica_and_the_summed_tokens():
    world, port = 2, 29500 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == pytest.approx(15.0)                       # the slowest rank's time, on every rank
        assert value == pytest.approx(2 * 256 / 15e-3)         # whole-job tokens/s: both replicas' tokens


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.job_throughput(100, 1, 50.0) == pytest.approx(2000.0)
