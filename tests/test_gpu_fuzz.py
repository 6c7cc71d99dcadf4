"""Seeded random structures against the oracle: grids, path subsets, sizes around tile and 16-byte
boundaries, weights with zeros, masks that empty whole modules, chunk sizes, kernel families,
tunings, rescaling, local levels and optimisers, all through the C ABI."""
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
         20000, 4096 * 5 + 8, 4096 * 3 + 1003]


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
    return K, numel, table, dtype, weights, reported, opts


@pytest.mark.parametrize("seed", range(64))
def test_random_structure_matches_the_oracle(seed):
    K, numel, table, dtype, weights, reported, opts = random_case(seed)
    cfg = synth.SyncConfig("fuzz%d" % seed, tuple(K), tuple(numel), dtype, momentum_std=1e-4, seed=seed)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1000 + seed)
    theta = torch.empty(cfg.module_params, device=DEV).normal_(0, 0.02, generator=gen)
    momentum = torch.empty(cfg.module_params, device=DEV).normal_(0, 1e-4, generator=gen)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    mod_off = np.concatenate([[0], np.cumsum([k * n for k, n in zip(K, numel)])])
    paths, keepalive = [], []
    for i in range(table.shape[0]):
        parts = [theta[int(mod_off[l]) + int(table[i, l]) * n:int(mod_off[l]) + (int(table[i, l]) + 1) * n]
                 + torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen) for l, n in enumerate(numel)]
        row = torch.cat(parts).to(tdt)
        if opts["misalign"]:                       # element-aligned only
            back = torch.empty(row.numel() + 4, dtype=tdt, device=DEV)
            view = back[1:1 + row.numel()]
            view.copy_(row)
            keepalive.append(back)
            row = view
        paths.append(row)
    pr = synth.SyncProblem(cfg, np.ascontiguousarray(table, dtype=np.int32), weights, reported, theta,
                           momentum, paths)
    before = host_state((theta, momentum, paths))

    code = B.DIPACO_BF16 if dtype == "bf16" else B.DIPACO_F32
    ctx = B.dipaco_create(K, numel, pr.table, weights, np.float32(0.7), np.float32(0.9), code,
                          opts["chunk"], 0)
    B.dipaco_set_kernel(ctx, opts["kernel"])
    try:
        B.dipaco_set_tuning(ctx, *opts["tuning"])
    except B.DipacoError as exc:                   # a layout that does not fit shared memory
        assert exc.status == B.DIPACO_EINVAL
    B.dipaco_set_module_scale(ctx, opts["scale"])
    B.dipaco_set_level_sync(ctx, opts["level_sync"])
    second = torch.empty_like(theta).normal_(0, 1e-4, generator=gen).abs_()
    v_host = helpers.tensor_to_numpy(second)
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
    B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths], reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)

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
