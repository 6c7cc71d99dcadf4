"""Seeded random structures against the oracle: grids, path subsets, sizes around tile and 16-byte
boundaries, weights with zeros, masks that empty whole modules, chunk sizes, kernel families,
tunings, rescaling, local levels and optimisers, and the way the synchronisation is carried out
(one call, the same call repeated on restored inputs, the chunk API with fresh write-back buffers,
host buffers, compact shards), all through the C ABI."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from paper_2403_10616_b200 import binding as B
from paper_2403_10616_b200 import synth
from tests import helpers
from tests.test_gpu_parity import assert_bf16_close, host_state

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
SIZES = [0, 1, 3, 7, 8, 9, 64, 1000, 2047, 2048, 2056, 4095, 4096, 4100, 4104, 8192, 8200, 12288 + 24,
         20000, 4096 * 5 + 8, 4096 * 3 + 1003, 3 * 8192 + 1003, 2 * 8192, 5 * 8192 + 24]


def random_case(seed):
    rng = np.random.RandomState(seed)
    L = int(rng.randint(1, 5))
    K = [int(rng.randint(1, 6)) for _ in range(L)]
    numel = [int(rng.choice(SIZES)) for _ in range(L)]
    if sum(numel) == 0:
        numel[0] = 4096 + 8
    full = synth.path_table(K)
    if rng.rand() < 0.4 and full.shape[0] > 2:      # a sampled subset of the paths
        keep = np.sort(rng.choice(full.shape[0], size=int(rng.randint(1, full.shape[0])), replace=False))
        table = full[keep]
    else:
        table = full
    P = table.shape[0]
    dtype = "bf16" if rng.rand() < 0.6 else "f32"
    weights = None
    if rng.rand() < 0.6:
        weights = rng.randint(0, 50, size=P).astype(np.float32)
        if rng.rand() < 0.5:
            weights[rng.randint(0, P)] = 0.0
    reported = None
    if rng.rand() < 0.6:
        reported = (rng.rand(P) > 0.35).astype(np.uint8)
    opts = {
        "chunk": int(rng.choice([0, 0, 1, 2, 3, 5, 32])),
        "kernel": int(rng.choice([B.DIPACO_KERNEL_AUTO, B.DIPACO_KERNEL_AUTO, B.DIPACO_KERNEL_VECTOR,
                                  B.DIPACO_KERNEL_SCALAR])),
        "tuning": [(0, 0, 0, 0), (1, 4, 1, 2), (2, 3, 1, 2), (1, 6, 2, 4), (1, 3, 4, 2), (3, 0, 1, 3)][
            int(rng.randint(0, 6))],
        "scale": rng.choice([0.5, 1.0, 2.0, 3.0], size=sum(K)).astype(np.float32) if rng.rand() < 0.4 else None,
        "level_sync": (rng.rand(L) > 0.3).astype(np.uint8) if rng.rand() < 0.3 else None,
        "optimizer": int(rng.choice([0, 0, 1, 2, 3])),
        "adam": (float(rng.choice([0.0, 0.5, 0.9])), float(rng.choice([0.0, 0.9, 0.999])), 1e-3,
                 float(rng.choice([0.0, 0.1])), int(rng.choice([0, 1, 7]))),
        "input_kind": int(rng.rand() < 0.25),
        "misalign": bool(rng.rand() < 0.2),
    }
    # drawn last, so the structures of the earlier seeds stay what they were
    opts["route"] = str(rng.choice(["one_call", "one_call", "repeat", "chunk_api", "host", "shards"]))
    opts["shards"] = int(rng.randint(2, 4))
    if opts["route"] in ("chunk_api", "host") and opts["chunk"] == 0:
        opts["chunk"] = int(rng.choice([1, 2, 5, 32]))
    if opts["route"] == "shards":
        opts["misalign"] = False
    return K, numel, table, dtype, weights, reported, opts


def configure(ctx, opts, second):
    """Apply the drawn options to a context; returns the oracle's Adam tuple (or None)."""
    B.dipaco_set_kernel(ctx, opts["kernel"])
    try:
        B.dipaco_set_tuning(ctx, *opts["tuning"])
    except B.DipacoError as exc:                   # a layout that does not fit shared memory
        assert exc.status == B.DIPACO_EINVAL
    B.dipaco_set_module_scale(ctx, opts["scale"])
    B.dipaco_set_level_sync(ctx, opts["level_sync"])
    adam = None
    if opts["optimizer"] == 3:
        b1, b2, eps, wd, step = opts["adam"]
        B.dipaco_set_adam(ctx, second.data_ptr(), b1, b2, eps, wd, step)
        f = lambda x: float(np.float32(x))
        adam = (f(b1), f(b2), f(eps), f(wd), 1 - f(b1) ** step if step else 1.0,
                1 - f(b2) ** step if step else 1.0)
    else:
        B.dipaco_set_optimizer(ctx, opts["optimizer"])
    B.dipaco_set_input_kind(ctx, opts["input_kind"])
    return adam


def run_route(ctx, opts, cfg, table, reported, theta, momentum, second, paths):
    """Carry the synchronisation out the drawn way, in place on the given tensors."""
    route = opts["route"]
    ptrs = [p.data_ptr() for p in paths]
    if route == "one_call":
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), ptrs, reported)
    elif route == "repeat":
        saved = (theta.clone(), momentum.clone(), second.clone(), [p.clone() for p in paths])
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), ptrs, reported)
        torch.cuda.synchronize()
        theta.copy_(saved[0]); momentum.copy_(saved[1]); second.copy_(saved[2])
        for p, q in zip(paths, saved[3]):
            p.copy_(q)
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), ptrs, reported)   # plan reused
    elif route == "chunk_api":
        chunk = opts["chunk"]
        nchunks, _ = B.dipaco_plan_chunks(ctx)
        B.dipaco_sync_begin(ctx, theta.data_ptr(), momentum.data_ptr(), reported)
        for c in range(nchunks):
            stage = [p.clone() for p in paths[c * chunk:(c + 1) * chunk]]
            B.dipaco_sync_accumulate(ctx, c, [p.data_ptr() for p in stage])
            torch.cuda.synchronize()
            del stage
        for c in range(nchunks):
            mine = paths[c * chunk:(c + 1) * chunk]
            if opts["level_sync"] is None:         # (levels kept local keep their contents)
                for p in mine:
                    p.fill_(float("nan"))          # write-back must not depend on the old contents
            B.dipaco_sync_writeback(ctx, c, [p.data_ptr() for p in mine])
        B.dipaco_sync_end(ctx)
    else:
        raise AssertionError(route)


@pytest.mark.parametrize("seed", range(96))
def test_random_structure_matches_the_oracle(seed):
    K, numel, table, dtype, weights, reported, opts = random_case(seed)
    cfg = synth.SyncConfig("fuzz%d" % seed, tuple(K), tuple(numel), dtype, momentum_std=1e-4, seed=seed)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1000 + seed)
    theta = torch.empty(cfg.module_params, device=DEV).normal_(0, 0.02, generator=gen)
    momentum = torch.empty(cfg.module_params, device=DEV).normal_(0, 1e-4, generator=gen)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    mod_off = np.concatenate([[0], np.cumsum([k * n for k, n in zip(K, numel)])])
    lvl_off = np.concatenate([[0], np.cumsum(numel)])
    paths, keepalive = [], []
    for i in range(table.shape[0]):
        parts = [theta[int(mod_off[l]) + int(table[i, l]) * n:int(mod_off[l]) + (int(table[i, l]) + 1) * n]
                 + torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen) for l, n in enumerate(numel)]
        row = torch.cat(parts).to(tdt)
        if opts["misalign"]:                       # element-aligned only, every path its own offset
            back = torch.empty(row.numel() + 8, dtype=tdt, device=DEV)
            off = 1 + i % 7
            view = back[off:off + row.numel()]
            view.copy_(row)
            keepalive.append(back)
            row = view
        paths.append(row)
    table = np.ascontiguousarray(table, dtype=np.int32)
    second = torch.empty_like(theta).normal_(0, 1e-4, generator=gen).abs_()
    v_host = helpers.tensor_to_numpy(second)
    before = host_state((theta, momentum, paths))
    code = B.DIPACO_BF16 if dtype == "bf16" else B.DIPACO_F32
    ctx = B.dipaco_create(K, numel, table, weights, np.float32(0.7), np.float32(0.9), code, opts["chunk"], 0)
    route = opts["route"]

    if route == "host":
        # everything lives in host memory (the path copies in one pinned block or one by one)
        theta, momentum, second = theta.cpu().pin_memory(), momentum.cpu().pin_memory(), second.cpu().pin_memory()
        if seed % 2:
            block = torch.stack([p.cpu() for p in paths]).pin_memory()
            paths = [block[i] for i in range(len(paths))]
        else:
            paths = [p.cpu() for p in paths]
        adam = configure(ctx, opts, second)
        B.dipaco_outer_sync_host(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths],
                                 reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    elif route == "shards":
        # S executors, each with its own packed slabs (Section 3.3); results put back side by side
        adam = configure(ctx, opts, second)
        S = opts["shards"]
        for s_idx in range(S):
            bounds = [B.dipaco_plan_shard(ctx, s_idx, S, l) for l in range(len(K))]
            mods = [slice(int(mod_off[l]) + e * numel[l] + bounds[l][0], int(mod_off[l]) + e * numel[l] + bounds[l][1])
                    for l in range(len(K)) for e in range(K[l])]
            lvls = [slice(int(lvl_off[l]) + bounds[l][0], int(lvl_off[l]) + bounds[l][1]) for l in range(len(K))]
            th_s = torch.cat([theta[sl] for sl in mods])
            mo_s = torch.cat([momentum[sl] for sl in mods])
            v_s = torch.cat([second[sl] for sl in mods])
            ps_s = [torch.cat([p[sl] for sl in lvls]) for p in paths]
            if th_s.numel() == 0:
                continue
            shard = B.dipaco_create_shard(ctx, s_idx, S, 0)
            if opts["optimizer"] == 3:
                B.dipaco_set_adam(shard, v_s.data_ptr(), *opts["adam"])
            B.dipaco_outer_sync(shard, th_s.data_ptr(), mo_s.data_ptr(), [p.data_ptr() for p in ps_s], reported)
            assert B.dipaco_device_status(shard) == B.DIPACO_OK
            B.dipaco_destroy(shard)
            pos = 0
            for sl in mods:
                n = sl.stop - sl.start
                theta[sl] = th_s[pos:pos + n]; momentum[sl] = mo_s[pos:pos + n]; second[sl] = v_s[pos:pos + n]
                pos += n
            for p, q in zip(paths, ps_s):
                pos = 0
                for sl in lvls:
                    n = sl.stop - sl.start
                    p[sl] = q[pos:pos + n]
                    pos += n
    else:
        adam = configure(ctx, opts, second)
        run_route(ctx, opts, cfg, table, reported, theta, momentum, second, paths)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    pr = synth.SyncProblem(cfg, table, weights, reported, theta, momentum, paths)



    scale64 = None if opts["scale"] is None else opts["scale"].astype(np.float64)
    want_th, want_mo, want_ps = helpers.run_oracle(cfg, pr.table, *before, weights, reported,
                                                   num_threads=4, module_scale=scale64,
                                                   level_sync=opts["level_sync"],
                                                   optimizer=opts["optimizer"],
                                                   second_moment=v_host if adam else None, adam=adam,
                                                   input_kind=opts["input_kind"])
    for got, want in ((helpers.tensor_to_numpy(theta), want_th), (helpers.tensor_to_numpy(momentum), want_mo),
                      (helpers.tensor_to_numpy(second), v_host)):
        err = np.abs(got.astype(np.float64) - want.astype(np.float64))
        assert np.all(err <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
    for p, want in zip(paths, want_ps):
        got = helpers.tensor_to_numpy(p)
        if dtype == "bf16":
            assert_bf16_close(got, want)
        else:
            err = np.abs(got.astype(np.float64) - want.astype(np.float64))
            assert np.all(err <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
