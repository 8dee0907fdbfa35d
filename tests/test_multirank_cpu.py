"""The N > 1 path of bench.py on CPU: two gloo ranks reduce their timings (max) and units (sum)."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t, u = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), dist)
    dist.barrier()
    out.put((rank, t, u))
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_units_by_sum():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 15.0, 3000.0), (1, 15.0, 3000.0)]


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.aggregate_over_ranks(3.0, 7.0, None) == (3.0, 7.0)
