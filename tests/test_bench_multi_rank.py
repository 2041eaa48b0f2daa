"""The N > 1 path of bench.py is "replicas only": the rotated step has no exchange between weight
matrices, so every rank runs the same workload and the only cross-rank logic is the reduction of the
measured times (maximum over ranks) and the scaling of the value by the number of replicas.  That
logic is exercised here on CPU with two gloo ranks."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [100.0 + 10.0 * rank, 50.0 - rank, 7.0, 3.0 * (rank + 1)]
        red = bench.max_over_ranks(mine, world, torch.device("cpu"), torch)
        out[rank] = (red, bench.replica_value(1000, world, red[0]))
    finally:
        dist.destroy_process_group()


def test_times_are_max_over_ranks_and_value_scales_with_replicas():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        out = mgr.dict()
        port = 29500 + os.getpid() % 2000
        procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        for r in range(2):
            red, value = out[r]
            assert red == [110.0, 50.0, 7.0, 6.0]
            assert value == pytest.approx(2 * 1000 / 0.110)


def test_single_rank_is_the_identity():
    import torch
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, torch.device("cpu"), torch) == [1.5, 2.5]
    assert bench.replica_value(10, 1, 1000.0) == 10.0
