"""World-size-2 check (gloo, CPU) of the benchmark's multi-replica bookkeeping: the reported time is
the maximum over ranks and the reported work is the sum over ranks."""
from __future__ import annotations

import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench.barrier(world)
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 1000.0 * (rank + 1), world, torch.device("cpu"))
    bench.barrier(world)
    out[rank] = (ms, units)
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_summed_units():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: (15.0, 3000.0), 1: (15.0, 3000.0)}


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(12.5, 7.0, 1, torch.device("cpu")) == (12.5, 7.0)
