"""The N > 1 path of bench.py shards nothing but the clock: every rank runs the same
per-GPU workload and only the timing is reduced (max over ranks).  Covered here with two
gloo ranks on the CPU."""
import os
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, l, w = bench.dist_setup(world, backend="gloo")
    bench.dist_barrier(w)
    secs = 0.010 * (rank + 1)          # rank 1 is the slow one
    value, t = bench.aggregate(1000, secs, w)
    q.put((rank, value, t))
    import torch.distributed as dist
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregate_is_total_rows_over_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29600 + os.getpid() % 300
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, t in res:
        assert t == pytest.approx(0.020)
        assert value == pytest.approx(2 * 1000 / 0.020)


def test_single_rank_aggregate():
    sys.path.insert(0, ROOT)
    import bench
    v, t = bench.aggregate(500, 0.5, 1)
    assert v == 1000 and t == 0.5
