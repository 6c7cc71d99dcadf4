"""World-size-2 checks (gloo, CPU) of the multi-rank bookkeeping.  Replicas: the reported time is
the maximum over ranks and the reported work is the sum over ranks.  Sharded executor (Section
3.3): the ranks' slabs tile every level exactly once and their planned traffic adds up to the
whole problem's, with no exchange other than this test's own gathering of the bounds."""
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


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2403_10616_b200 import binding as B
    from paper_2403_10616_b200 import build as libbuild
    from paper_2403_10616_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    libbuild.build()
    cfg = synth.CONFIGS["grid16x16-masked"]
    reported = synth.reported_mask(cfg)
    # every rank plans from the same description of the whole problem: no device, no data
    whole = B.dipaco_create(cfg.modules_per_level, cfg.level_numel, synth.path_table(cfg.modules_per_level),
                            synth.path_weights(cfg), cfg.outer_lr, cfg.outer_momentum, B.DIPACO_BF16, 0,
                            device=-1)
    bounds = [B.dipaco_plan_shard(whole, rank, world, l) for l in range(cfg.num_levels)]
    mine = B.dipaco_create_shard(whole, rank, world, device=-1)
    traffic = B.dipaco_plan_traffic(mine, reported)[0]
    total = B.dipaco_plan_traffic(whole, reported)[0]
    B.dipaco_destroy(mine)
    B.dipaco_destroy(whole)
    t = torch.tensor([b for ab in bounds for b in ab] + [traffic, total], dtype=torch.int64)
    gathered = [torch.zeros_like(t) for _ in range(world)]
    dist.all_gather(gathered, t)
    out[rank] = [g.tolist() for g in gathered]
    dist.destroy_process_group()


def test_two_ranks_split_one_problem_into_slabs_that_tile_it():
    from paper_2403_10616_b200 import synth
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
        seen = dict(out)
    assert seen[0] == seen[1]
    cfg = synth.CONFIGS["grid16x16-masked"]
    rows = seen[0]
    for l, n in enumerate(cfg.level_numel):
        cuts = [(rows[r][2 * l], rows[r][2 * l + 1]) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))      # every element owned exactly once
        assert all(a < b for a, b in cuts)
    traffic = [rows[r][-2] for r in range(world)]
    assert sum(traffic) == rows[0][-1]
    assert abs(traffic[0] - traffic[1]) < 0.001 * rows[0][-1]
