"""CPU tests of the CUDA library's host side: exported symbols, validation, and planning (the
contributor sets and coefficients).

No compute call is made: contexts are created plan-only (device = -1)."""
from __future__ import annotations

import ctypes
import os
import re

import numpy as np
import pytest

from paper_2403_10616_b200 import binding as B
from paper_2403_10616_b200 import build as libbuild
from paper_2403_10616_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    libbuild.build()
    B.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dipaco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dipaco_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.LIB_PATH)
    names = declared_functions()
    assert "dipaco_create" in names and "dipaco_outer_sync" in names and "dipaco_destroy" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == names


def test_strerror_names_every_status():
    for code in (0, -1, -2, -3, -4, -5, -6, -7):
        assert B.strerror(code) != "unknown status"
    assert B.strerror(-99) == "unknown status"


def plan_ctx(cfg, table=None, weights=None, chunk_paths=0):
    table = synth.path_table(cfg.modules_per_level) if table is None else table
    code = B.DIPACO_BF16 if cfg.path_dtype == "bf16" else B.DIPACO_F32
    return B.dipaco_create(cfg.modules_per_level, cfg.level_numel, table, weights,
                           cfg.outer_lr, cfg.outer_momentum, code, chunk_paths, device=-1)


def test_plan_only_context_refuses_compute_calls():
    cfg = synth.CONFIGS["grid2x2"]
    ctx = plan_ctx(cfg)
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_outer_sync(ctx, 16, 16, [16] * cfg.num_paths, None, stream=0)
    assert e.value.status == B.DIPACO_ENODEV
    assert B.dipaco_device_status(ctx) == B.DIPACO_ENODEV
    B.dipaco_destroy(ctx)


@pytest.mark.parametrize("bad", ["entry", "negative_entry", "levels", "weights_nan", "weights_neg",
                                 "k_zero", "n_negative", "lr_inf", "dtype"])
def test_create_rejects_invalid_arguments(bad):
    K = np.array([1, 2, 2], dtype=np.int32)
    N = np.array([8, 8, 8], dtype=np.int64)
    table = synth.path_table(K).copy()
    w = np.ones(4, dtype=np.float32)
    lr, dtype = 0.7, B.DIPACO_F32
    if bad == "entry":
        table[2, 1] = 2
    elif bad == "negative_entry":
        table[0, 0] = -1
    elif bad == "weights_nan":
        w[1] = np.nan
    elif bad == "weights_neg":
        w[1] = -1.0
    elif bad == "k_zero":
        K[2] = 0
    elif bad == "n_negative":
        N[0] = -5
    elif bad == "lr_inf":
        lr = float("inf")
    elif bad == "dtype":
        dtype = 7
    if bad == "levels":
        lib = B.load()
        h = ctypes.c_void_p()
        rc = lib.dipaco_create(ctypes.byref(h), 0, K.ctypes.data, N.ctypes.data, 4, table.ctypes.data,
                               None, 0.7, 0.9, 0, 0, -1)
        assert rc == B.DIPACO_EINVAL and not h.value
        return
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_create(K, N, table, w, lr, 0.9, dtype, 0, device=-1)
    assert e.value.status == B.DIPACO_EINVAL


def test_toy_grid_contributor_sets_match_the_papers_figure():
    cfg = synth.CONFIGS["grid2x2"]
    ctx = plan_ctx(cfg)
    want = {(0, 0): [0, 1, 2, 3], (1, 0): [0, 1], (1, 1): [2, 3], (2, 0): [0, 2], (2, 1): [1, 3]}
    for (l, e), paths in want.items():
        members, contributors, coeff, upd = B.dipaco_plan_module(ctx, l, e, cfg.num_paths)
        assert members.tolist() == paths and contributors.tolist() == paths and upd
        np.testing.assert_array_equal(coeff, np.full(len(paths), 1.0 / len(paths), np.float32))
    B.dipaco_destroy(ctx)


def test_coefficients_are_normalised_per_module_over_reporting_paths():
    cfg = synth.CONFIGS["grid16x16-masked"].scaled((16, 16, 16))
    w = synth.path_weights(cfg)
    r = synth.reported_mask(cfg)
    table = synth.path_table(cfg.modules_per_level)
    ctx = plan_ctx(cfg, table, w)
    for l in range(3):
        for e in range(cfg.modules_per_level[l]):
            members, contributors, coeff, upd = B.dipaco_plan_module(ctx, l, e, cfg.num_paths, r)
            S = [i for i in range(cfg.num_paths) if table[i, l] == e]
            R = [i for i in S if r[i]]
            assert members.tolist() == S and contributors.tolist() == R and upd
            total = np.sum(w[R].astype(np.float64))
            np.testing.assert_array_equal(coeff, (w[R].astype(np.float64) / total).astype(np.float32))
            assert abs(float(np.sum(coeff.astype(np.float64))) - 1.0) < 1e-6
    # a module whose paths are all masked, and zero total weight
    r2 = r.copy()
    r2[[i for i in range(cfg.num_paths) if table[i, 1] == 3]] = 0
    members, contributors, coeff, upd = B.dipaco_plan_module(ctx, 1, 3, cfg.num_paths, r2)
    assert len(members) == 16 and len(contributors) == 0 and not upd
    w0 = w.copy()
    w0[[i for i in range(cfg.num_paths) if table[i, 2] == 5]] = 0.0
    B.dipaco_set_weights(ctx, w0)
    _, contributors, _, upd = B.dipaco_plan_module(ctx, 2, 5, cfg.num_paths, None)
    assert len(contributors) == 0 and not upd
    B.dipaco_set_weights(ctx, None)
    _, contributors, coeff, upd = B.dipaco_plan_module(ctx, 2, 5, cfg.num_paths, None)
    assert upd and np.all(coeff == np.float32(1 / 16))
    B.dipaco_destroy(ctx)


def test_offsets_follow_level_module_element_order():
    cfg = synth.CONFIGS["grid4x4x4x4"].scaled((7, 5, 3, 11, 2))
    ctx = plan_ctx(cfg)
    theta_off = 0
    path_off = 0
    for l, (k, n) in enumerate(zip(cfg.modules_per_level, cfg.level_numel)):
        for e in range(k):
            assert B.dipaco_plan_offsets(ctx, l, e) == (theta_off, path_off, n)
            theta_off += n
        path_off += n
    with pytest.raises(B.DipacoError):
        B.dipaco_plan_offsets(ctx, 1, 4)
    B.dipaco_destroy(ctx)


def test_arbitrary_subset_of_paths_and_unused_modules():
    """Any path set is allowed (path sampling); a module nobody uses has no members."""
    K, N = (1, 3, 3), (4, 4, 4)
    table = np.array([[0, 0, 1], [0, 2, 1], [0, 2, 2]], dtype=np.int32)
    ctx = B.dipaco_create(K, N, table, None, 0.7, 0.9, B.DIPACO_F32, 0, device=-1)
    members, contributors, _, upd = B.dipaco_plan_module(ctx, 1, 1, 3)
    assert len(members) == 0 and len(contributors) == 0 and not upd
    members, _, coeff, _ = B.dipaco_plan_module(ctx, 1, 2, 3)
    assert members.tolist() == [1, 2] and coeff.tolist() == [0.5, 0.5]
    B.dipaco_destroy(ctx)


def test_chunk_count_and_scratch_size():
    cfg = synth.CONFIGS["grid16x16"].scaled((1000, 1001, 1002))
    ctx = plan_ctx(cfg, chunk_paths=32)
    n, scratch = B.dipaco_plan_chunks(ctx)
    # shared level and the 16 level-2 modules span chunks; level-1 modules live inside one chunk.
    # A module's slot starts where its theta starts within a group of eight elements and slots
    # do not share such a group: at most 14 elements of padding per module.
    need = 1000 + 16 * 1002
    assert n == 8 and need <= scratch <= need + 17 * 14 and scratch % 8 == 0
    B.dipaco_destroy(ctx)
    # sizes that are multiples of eight need no padding at all
    even = synth.CONFIGS["grid16x16"].scaled((1000, 1008, 1016))
    ctx = plan_ctx(even, chunk_paths=32)
    assert B.dipaco_plan_chunks(ctx) == (8, 1000 + 16 * 1016)
    B.dipaco_destroy(ctx)
    ctx = plan_ctx(cfg, chunk_paths=0)
    assert B.dipaco_plan_chunks(ctx) == (1, 0)
    B.dipaco_destroy(ctx)
    ctx = plan_ctx(cfg, chunk_paths=100)
    assert B.dipaco_plan_chunks(ctx)[0] == 3
    B.dipaco_destroy(ctx)


@pytest.mark.parametrize("name,numel,ctas", [("grid16x16", (50_000_000,) * 3, 296),
                                             ("grid4x4x4x4", (20_000_000,) + (10_000_000,) * 4, 148),
                                             ("grid2x2", (16384, 65536, 65536), 296),
                                             ("grid4x4", (4096 + 17, 2048 * 3, 100), 7)])
def test_split_covers_every_full_tile_once_and_balances_cost(name, numel, ctas):
    cfg = synth.CONFIGS[name].scaled(numel)
    tile = 2048
    ctx = plan_ctx(cfg)
    lvl, mod, beg, end, first = B.dipaco_plan_split(ctx, ctas, tile)
    assert first[0] == 0 and first[-1] == len(lvl) and np.all(np.diff(first) >= 0)
    assert np.all(beg % tile == 0) and np.all(end % tile == 0) and np.all(end > beg)
    covered = {}
    for l, e, b, t in zip(lvl, mod, beg, end):
        covered.setdefault((int(l), int(e)), []).append((int(b), int(t)))
    for l, (k, n) in enumerate(zip(cfg.modules_per_level, cfg.level_numel)):
        full = n // tile * tile
        for e in range(k):
            spans = sorted(covered.get((l, e), []))
            pos = 0
            for b, t in spans:
                assert b == pos
                pos = t
            assert pos == full
    # bytes per element: theta r/w + momentum r/w + contributors read + members written
    s = 2 if cfg.path_dtype == "bf16" else 4
    per_level = [16 + 2 * s * (cfg.num_paths // k) for k in cfg.modules_per_level]
    cost = np.zeros(ctas)
    for b in range(ctas):
        for i in range(first[b], first[b + 1]):
            cost[b] += per_level[lvl[i]] * (end[i] - beg[i])
    heaviest_tile = max(per_level) * tile
    assert cost.max() - cost.sum() / ctas <= 1.01 * heaviest_tile
    B.dipaco_destroy(ctx)


def test_planned_traffic_of_resident_mode_is_the_algorithmic_minimum():
    for name in ("grid16x16", "grid16x16-masked", "grid4x4x4x4", "grid4x4"):
        cfg = synth.CONFIGS[name]
        r = synth.reported_mask(cfg)
        ctx = plan_ctx(cfg, weights=synth.path_weights(cfg))
        nbytes, launches = B.dipaco_plan_traffic(ctx, r)
        assert launches == 1 and nbytes == synth.algorithmic_bytes(cfg, r)
        B.dipaco_destroy(ctx)
    # Walking the 16x16 workload in chunks of 32 paths: one launch per chunk.  On top of the
    # algorithmic bytes every launch but the last reads theta again and carries the fp32 partial
    # sum of the modules whose paths span chunks (the shared block and the 16 last-level modules:
    # 850e6 parameters): theta re-read 7 times, partial written 7 times and read 7 times.
    cfg = synth.CONFIGS["grid16x16"]
    ctx = plan_ctx(cfg, chunk_paths=32)
    nbytes, launches = B.dipaco_plan_traffic(ctx)
    spanning = 17 * 50_000_000
    assert launches == 8
    assert nbytes == synth.algorithmic_bytes(cfg) + spanning * 4 * (7 + 7 + 7)
    assert nbytes < 252e9
    B.dipaco_destroy(ctx)
    # a module that nobody updates is refilled inside the first launch: no extra launch
    cfg = synth.CONFIGS["grid16x16-masked"]
    ctx = plan_ctx(cfg, chunk_paths=32, weights=synth.path_weights(cfg))
    r = synth.reported_mask(cfg).copy()
    r[[i for i in range(256) if synth.path_table(cfg.modules_per_level)[i, 1] == 3]] = 0
    nbytes, launches = B.dipaco_plan_traffic(ctx, r)
    assert launches == 8
    B.dipaco_destroy(ctx)


def test_shards_partition_the_planned_traffic():
    cfg = synth.CONFIGS["grid16x16"]
    ctx = plan_ctx(cfg)
    whole, _ = B.dipaco_plan_traffic(ctx)
    parts = []
    for shard in range(8):
        B.dipaco_set_shard(ctx, shard, 8)
        parts.append(B.dipaco_plan_traffic(ctx)[0])
    assert sum(parts) == whole
    assert max(parts) - min(parts) < 0.001 * whole     # equal slabs up to the 8192-element grain
    for bad in ((8, 8), (-1, 8), (0, 0)):
        with pytest.raises(B.DipacoError):
            B.dipaco_set_shard(ctx, *bad)
    B.dipaco_destroy(ctx)


def test_tuning_setters_validate_their_arguments():
    ctx = plan_ctx(synth.CONFIGS["grid2x2"], chunk_paths=2)
    for good in ((0, 0), (1 << 20, 32), (0, 4096)):
        B.dipaco_set_work_items(ctx, *good)
    for bad in ((-1, 0), (0, -1), (0, 5000)):
        with pytest.raises(B.DipacoError) as e:
            B.dipaco_set_work_items(ctx, *bad)
        assert e.value.status == B.DIPACO_EINVAL
    for good in (-1, 0, 1, 16):
        B.dipaco_set_host_threads(ctx, good)
    for bad in (-2, 1000):
        with pytest.raises(B.DipacoError):
            B.dipaco_set_host_threads(ctx, bad)
    for good in (0, 1 << 20, 1 << 33):
        B.dipaco_set_host_unit_bytes(ctx, good)
    with pytest.raises(B.DipacoError):
        B.dipaco_set_host_unit_bytes(ctx, -5)
    # the diagnostic needs a device
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_selftest_wait_expiry(ctx, 1000, stream=0)
    assert e.value.status == B.DIPACO_ENODEV
    B.dipaco_destroy(ctx)


def test_compact_shard_contexts_tile_the_problem_exactly_once():
    """dipaco_plan_shard / dipaco_create_shard (Section 3.3, sharded executor): over the shards
    every element of every level is owned exactly once, a shard context is the same grid with the
    slab sizes as module sizes, and the planned traffic of the shards sums to the whole's."""
    cfg = synth.CONFIGS["grid16x16-masked"].scaled((100_003, 8192 * 5, 8191))
    w = synth.path_weights(cfg)
    r = synth.reported_mask(cfg)
    whole = plan_ctx(cfg, weights=w)
    total, _ = B.dipaco_plan_traffic(whole, r)
    S = 3
    parts = 0
    for l, n in enumerate(cfg.level_numel):
        cuts = [B.dipaco_plan_shard(whole, s, S, l) for s in range(S)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n
        for (a0, b0), (a1, b1) in zip(cuts, cuts[1:]):
            assert b0 == a1 and a0 <= b0 and a1 <= b1
        assert all(a % 8192 == 0 for a, _ in cuts)
    for s in range(S):
        ctx = B.dipaco_create_shard(whole, s, S, device=-1)
        for l in range(cfg.num_levels):
            a, b = B.dipaco_plan_shard(whole, s, S, l)
            for e in (0, cfg.modules_per_level[l] - 1):
                _, _, numel = B.dipaco_plan_offsets(ctx, l, e)
                assert numel == b - a
        # same contributor sets and coefficients as the whole problem
        for (l, e) in ((0, 0), (1, 5), (2, 15)):
            got = B.dipaco_plan_module(ctx, l, e, cfg.num_paths, r)
            want = B.dipaco_plan_module(whole, l, e, cfg.num_paths, r)
            for x, y in zip(got[:3], want[:3]):
                np.testing.assert_array_equal(x, y)
        parts += B.dipaco_plan_traffic(ctx, r)[0]
        B.dipaco_destroy(ctx)
    assert parts == total
    with pytest.raises(B.DipacoError):
        B.dipaco_create_shard(whole, 3, 3, device=-1)
    with pytest.raises(B.DipacoError):
        B.dipaco_plan_shard(whole, 0, 3, 7)
    B.dipaco_destroy(whole)


def test_a_c99_program_can_use_the_library(tmp_path):
    """The header compiles as C and a plain C caller links against the shared library."""
    import subprocess
    exe = str(tmp_path / "plan_from_c")
    src = os.path.join(ROOT, "tests", "c", "plan_from_c.c")
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), src,
                           "-o", exe, "-L", libdir, "-ldipaco", "-Wl,-rpath," + libdir])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr
