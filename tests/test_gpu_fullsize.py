"""Parity at the benchmark's full sizes, in the launch configurations bench.py times.

Workloads: the 16x16 grid (256 paths, 150M parameters per path, bf16), the same with 20 % of the
paths not reporting and Zipf weights, the 4x4x4x4 grid (256 paths, 60M parameters per path,
1 % of the deltas a hundred times larger), and the 16x16 grid with an odd level size (20,000,003:
modules and slots inside 16-byte units, the kernel variant for shifted buffers).  Legs: resident one-pass (default kernel and tuning),
the chunk walk (chunks of 32 paths) and the host-buffer entry point.

The oracle cannot run 38.4e9 path elements in test time; elements are independent, so it is
evaluated on sampled element indices (first and last 65,536 of every module plus 2^20 seeded
random ones per level), gathered from the device buffers before the call.  Whole-tensor
properties are checked on the device: every copy equals cast(theta') of its module, a second run
from regenerated inputs gives bitwise the same result, and the other legs give bitwise the
resident result (order-independent integer checksums of every buffer).
"""
from __future__ import annotations

import gc

import numpy as np
import pytest
import torch

from paper_2403_10616_b200 import binding as B
from paper_2403_10616_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def checksums(theta, momentum, paths, piece=50_000_000):
    """Order-independent integer checksums (sum of the bit patterns) of every buffer."""
    def total(t, bits):
        flat = t.view(bits)
        acc = 0
        for start in range(0, flat.numel(), piece):
            acc += int(flat[start:start + piece].to(torch.int64).sum().item())
        return acc
    out = [total(theta, torch.int32), total(momentum, torch.int32)]
    out.extend(total(p, torch.int16) for p in paths)
    return out


def free_device_memory():
    gc.collect()
    torch.cuda.empty_cache()
    return torch.cuda.mem_get_info()[0]


def run_on_device(problem, chunk_paths):
    sync = B.OuterSync.for_problem(problem, chunk_paths=chunk_paths)
    sync.sync(problem.theta, problem.momentum, problem.paths, problem.reported)
    assert sync.status() == B.DIPACO_OK
    sync.close()


class Sampler:
    """Sampled element indices of every level, and the gathers that turn the full problem into
    the small problem the oracle is run on (same grid, level sizes = number of samples)."""

    def __init__(self, problem, seed=1234, windows=()):
        cfg = problem.cfg
        gen = torch.Generator(device=DEV)
        gen.manual_seed(seed)
        self.cfg = cfg
        self.idx = []
        for n in cfg.level_numel:
            edge = min(65536, n)
            parts = [torch.arange(0, edge, device=DEV), torch.arange(n - edge, n, device=DEV),
                     torch.randint(0, n, (1 << 20,), device=DEV, generator=gen)]
            # extra windows of consecutive indices (clipped to the level), e.g. around 2^31
            parts.extend(torch.arange(max(a, 0), min(b, n), device=DEV) for a, b in windows if a < n)
            self.idx.append(torch.cat(parts))
        self.small = cfg.scaled(tuple(int(i.numel()) for i in self.idx))
        self.mod_off = problem.module_offsets()
        self.lvl_off = problem.level_offsets()

    def modules(self, t):
        parts = []
        for l, k in enumerate(self.cfg.modules_per_level):
            n = self.cfg.level_numel[l]
            for e in range(k):
                base = int(self.mod_off[l]) + e * n
                parts.append(t[base:base + n][self.idx[l].to(t.device)])
        return helpers.tensor_to_numpy(torch.cat(parts))

    def path(self, p):
        parts = [p[int(self.lvl_off[l]):int(self.lvl_off[l]) + n][self.idx[l].to(p.device)]
                 for l, n in enumerate(self.cfg.level_numel)]
        return helpers.tensor_to_numpy(torch.cat(parts))

    def inputs(self, problem):
        return (self.modules(problem.theta), self.modules(problem.momentum),
                [self.path(p) for p in problem.paths])

    def expected(self, problem, before):
        return helpers.run_oracle(self.small, problem.table, *before, problem.weights,
                                  problem.reported, num_threads=16)

    def check(self, theta, momentum, paths, want, every=5):
        want_th, want_mo, want_ps = want
        for got, exp in ((self.modules(theta), want_th), (self.modules(momentum), want_mo)):
            err = np.abs(got.astype(np.float64) - exp.astype(np.float64))
            assert np.all(err <= 1e-6 * (1.0 + np.abs(exp.astype(np.float64))))
        for i in range(0, len(paths), every):
            helpers.assert_bf16_copies_close(self.path(paths[i]), want_ps[i], "copy of path %d" % i)


def assert_every_copy_is_the_cast_of_its_module(problem):
    cfg = problem.cfg
    mod_off, lvl_off = problem.module_offsets(), problem.level_offsets()
    for l, k in enumerate(cfg.modules_per_level):
        n = cfg.level_numel[l]
        for e in range(k):
            base = int(mod_off[l]) + e * n
            want = problem.theta[base:base + n].to(torch.bfloat16).view(torch.int16)
            for i in range(cfg.num_paths):
                if problem.table[i, l] == e:
                    slot = problem.paths[i][int(lvl_off[l]):int(lvl_off[l]) + n].view(torch.int16)
                    assert torch.equal(slot, want)


@pytest.mark.parametrize("name", ["grid16x16", "grid16x16-masked", "grid4x4x4x4", "grid16x16-odd-level-size"])
def test_full_size_sampled_parity_properties_and_reproducibility(name):
    cfg = synth.CONFIGS[name]
    need = cfg.path_params * 2 + 8 * cfg.module_params
    if free_device_memory() < need * 1.03 + 8e9:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    pr = synth.make_problem(cfg, DEV)
    sampler = Sampler(pr)
    before = sampler.inputs(pr)
    run_on_device(pr, 0)
    torch.cuda.synchronize()
    want = sampler.expected(pr, before)
    sampler.check(pr.theta, pr.momentum, pr.paths, want)
    assert_every_copy_is_the_cast_of_its_module(pr)
    first = checksums(pr.theta, pr.momentum, pr.paths)
    del pr
    free_device_memory()

    # a second run from regenerated inputs: bitwise the same
    again = synth.make_problem(cfg, DEV)
    run_on_device(again, 0)
    torch.cuda.synchronize()
    assert checksums(again.theta, again.momentum, again.paths) == first
    del again
    free_device_memory()

    # the chunk walk that bench.py times on this workload (chunks of 32 paths): bitwise the
    # resident result, and checked against the oracle's samples in its own right
    if cfg.chunk_paths > 0:
        chunked = synth.make_problem(cfg, DEV)
        run_on_device(chunked, cfg.chunk_paths)
        torch.cuda.synchronize()
        sampler.check(chunked.theta, chunked.momentum, chunked.paths, want)
        assert checksums(chunked.theta, chunked.momentum, chunked.paths) == first
        del chunked
        free_device_memory()


def test_host_buffer_entry_point_at_scale_matches_the_oracle_and_the_resident_result():
    """dipaco_outer_sync_host, the call behind bench.py's end-to-end number, on the 16x16 grid with
    20M parameters per level (256 paths of 60M parameters: 30.7 GB of bf16 copies in pinned host
    memory, Zipf weights, 20 % of the paths not reporting): sampled against the oracle and bitwise
    equal to the resident result of the same inputs."""
    cfg = synth.CONFIGS["grid16x16-masked"].scaled((20_000_000,) * 3, name="grid16x16-masked-20M")
    need = cfg.path_params * 2 + 8 * cfg.module_params
    if free_device_memory() < need * 1.03 + 12e9:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    try:
        with open("/proc/meminfo") as f:
            avail = [int(line.split()[1]) * 1024 for line in f if line.startswith("MemAvailable:")][0]
    except (OSError, IndexError):
        avail = None
    if avail is not None and avail < need * 1.5:
        pytest.skip("needs %.0f GB of pinned host memory" % (need / 1e9))
    pr = synth.make_problem(cfg, DEV)
    table, weights, reported = pr.table, pr.weights, pr.reported
    sampler = Sampler(pr)
    before = sampler.inputs(pr)
    want = sampler.expected(pr, before)
    # the same inputs in pinned host memory
    theta_h = torch.empty(cfg.module_params, dtype=torch.float32, pin_memory=True)
    mom_h = torch.empty(cfg.module_params, dtype=torch.float32, pin_memory=True)
    paths_h = torch.empty((cfg.num_paths, cfg.params_per_path), dtype=torch.bfloat16, pin_memory=True)
    theta_h.copy_(pr.theta)
    mom_h.copy_(pr.momentum)
    paths_h.copy_(pr.storage)
    torch.cuda.synchronize()
    # resident reference on the device copy
    run_on_device(pr, 0)
    torch.cuda.synchronize()
    sampler.check(pr.theta, pr.momentum, pr.paths, want)
    resident = checksums(pr.theta, pr.momentum, pr.paths)
    del pr
    free_device_memory()

    code = B.DIPACO_BF16
    ctx = B.dipaco_create(cfg.modules_per_level, cfg.level_numel, table, weights,
                          np.float32(cfg.outer_lr), np.float32(cfg.outer_momentum), code, 32, 0)
    rows = [paths_h[i] for i in range(cfg.num_paths)]
    B.dipaco_outer_sync_host(ctx, theta_h.data_ptr(), mom_h.data_ptr(), [r.data_ptr() for r in rows],
                             reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    free_device_memory()
    sampler.check(theta_h, mom_h, rows, want)
    theta_d, mom_d, paths_d = theta_h.to(DEV), mom_h.to(DEV), paths_h.to(DEV)
    assert checksums(theta_d, mom_d, [paths_d[i] for i in range(cfg.num_paths)]) == resident


@pytest.mark.parametrize("kernel", ["auto", "vector"])
def test_a_module_with_more_than_2_pow_31_parameters(kernel):
    """The largest sizes: one module of 2^31 + 12,293 parameters shared by two paths (bf16), next
    to a level of two small modules.  Element indices, byte offsets into the copies (4.3 GB each)
    and the partial-sum scratch all pass 2^31 and 2^32; the module's last five parameters do not
    fill a 16-byte unit, so the one-element-per-thread kernel runs beyond 2^31 too.  Sampled
    against the oracle with extra windows on both sides of 2^31 and of 2^32 bytes; the chunk walk
    (one path per chunk, so the big module carries a partial sum) must give bitwise the same."""
    big = (1 << 31) + 3 * 4096 + 5
    cfg = synth.SyncConfig("one-huge-module", (1, 2), (big, 4099), "bf16", weights="tokens",
                           momentum_std=1e-4)
    need = cfg.path_params * 2 + 8 * cfg.module_params
    # the generator holds two fp32 temporaries of the module's size besides the problem itself
    if free_device_memory() < need + 3 * 4 * big + 8e9:
        pytest.skip("needs %.0f GB of free device memory" % ((need + 12 * big) / 1e9))
    code = {"auto": B.DIPACO_KERNEL_AUTO, "vector": B.DIPACO_KERNEL_VECTOR}[kernel]

    def run(problem, chunk_paths):
        sync = B.OuterSync.for_problem(problem, chunk_paths=chunk_paths)
        B.dipaco_set_kernel(sync.ctx, code)
        sync.sync(problem.theta, problem.momentum, problem.paths, problem.reported)
        assert sync.status() == B.DIPACO_OK
        sync.close()
        torch.cuda.synchronize()

    pr = synth.make_problem(cfg, DEV)
    free_device_memory()
    half = 1 << 30   # element whose byte offset inside a bf16 copy is 2^31; fp32 offset 2^32
    sampler = Sampler(pr, windows=[(half - 8192, half + 8192), ((1 << 31) - 8192, big)])
    before = sampler.inputs(pr)
    run(pr, 0)
    want = sampler.expected(pr, before)
    sampler.check(pr.theta, pr.momentum, pr.paths, want, every=1)
    assert_every_copy_is_the_cast_of_its_module(pr)
    first = checksums(pr.theta, pr.momentum, pr.paths)
    del pr
    free_device_memory()

    chunked = synth.make_problem(cfg, DEV)
    free_device_memory()
    run(chunked, 1)
    assert checksums(chunked.theta, chunked.momentum, chunked.paths) == first
    del chunked
    free_device_memory()
