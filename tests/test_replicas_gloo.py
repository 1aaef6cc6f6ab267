"""The multi-GPU path is replicas only (no exchange on the data path): what the ranks share is the timing
reduction of the benchmark. Exercised here on CPU with two gloo ranks."""
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
    try:
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        worst = bench.max_over_ranks(local_ms)
        q.put((rank, worst, bench.replica_value(worst, gamma=7, world=world)))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_replica_value_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, value in got:
        assert worst == 15.0                               # every rank sees the slowest rank's time
        assert abs(value - 15.0 * 1e3 / 14 / 2) < 1e-9     # two replicas: twice the draft steps in that time


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.replica_value(14.0, gamma=7, world=1) == 1000.0
