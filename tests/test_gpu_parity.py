"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Tolerance (fp32 results theta', m'): |gpu - oracle| <= 1e-6 * (1 + |oracle|).  Path copies must
equal cast(gpu theta') bit for bit (fp32: the value itself; bf16: round-to-nearest-even) and, for
bf16, lie within one bf16 step (the exact spacing at the expected value) plus the fp32 tolerance
of the oracle's copy (helpers.assert_bf16_copies_close).  Kernel families, resident and chunked
mode and repeated runs must agree bitwise.
"""
from __future__ import annotations

import ctypes

import numpy as np
import pytest
import torch

from paper_2403_10616_b200 import binding as B
from paper_2403_10616_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def clone_problem(pr):
    return (pr.theta.clone(), pr.momentum.clone(), [p.clone() for p in pr.paths])


def make_ctx(pr, chunk_paths=0, kernel=B.DIPACO_KERNEL_AUTO, weights="cfg"):
    cfg = pr.cfg
    code = B.DIPACO_BF16 if cfg.path_dtype == "bf16" else B.DIPACO_F32
    w = pr.weights if isinstance(weights, str) else weights
    ctx = B.dipaco_create(cfg.modules_per_level, cfg.level_numel, pr.table, w,
                          np.float32(cfg.outer_lr), np.float32(cfg.outer_momentum), code,
                          chunk_paths, 0)
    B.dipaco_set_kernel(ctx, kernel)
    return ctx


def run_gpu(pr, state, reported="cfg", chunk_paths=0, kernel=B.DIPACO_KERNEL_AUTO, weights="cfg",
            tuning=None):
    theta, momentum, paths = state
    ctx = make_ctx(pr, chunk_paths, kernel, weights)
    if tuning:
        B.dipaco_set_tuning(ctx, *tuning)
    r = pr.reported if isinstance(reported, str) else reported
    B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths], r)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    launches = B.dipaco_launch_count(ctx)
    B.dipaco_destroy(ctx)
    return launches


def assert_matches_oracle(pr, before, after, reported="cfg", weights="cfg", threads=8):
    cfg = pr.cfg
    th0, mo0, ps0 = before
    r = pr.reported if isinstance(reported, str) else reported
    w = pr.weights if isinstance(weights, str) else weights
    want_th, want_mo, want_ps = helpers.run_oracle(cfg, pr.table, th0, mo0, ps0, w, r,
                                                   num_threads=threads)
    got_th = helpers.tensor_to_numpy(after[0])
    got_mo = helpers.tensor_to_numpy(after[1])
    for got, want, name in ((got_th, want_th, "theta"), (got_mo, want_mo, "momentum")):
        err = np.abs(got.astype(np.float64) - want.astype(np.float64))
        bound = 1e-6 * (1.0 + np.abs(want.astype(np.float64)))
        assert np.all(err <= bound), "%s max err %g" % (name, float((err / bound).max()))
    lvl = pr.level_offsets()
    mod = pr.module_offsets()
    for i, p in enumerate(after[2]):
        got = helpers.tensor_to_numpy(p)
        for l in range(cfg.num_levels):
            n = cfg.level_numel[l]
            src = int(mod[l]) + int(pr.table[i, l]) * n
            slot = got[int(lvl[l]):int(lvl[l]) + n]
            if cfg.path_dtype == "bf16":
                np.testing.assert_array_equal(slot, helpers.float_to_bf16_bits_torch(got_th[src:src + n]))
                assert_bf16_close(slot, want_ps[i][int(lvl[l]):int(lvl[l]) + n])
            else:
                np.testing.assert_array_equal(slot.view(np.uint32), got_th[src:src + n].view(np.uint32))


def assert_bf16_close(got_bits, want_bits):
    helpers.assert_bf16_copies_close(got_bits, want_bits)


def assert_states_bitwise_equal(a, b):
    assert torch.equal(a[0].view(torch.int32), b[0].view(torch.int32))
    assert torch.equal(a[1].view(torch.int32), b[1].view(torch.int32))
    for x, y in zip(a[2], b[2]):
        bits = torch.int16 if x.dtype == torch.bfloat16 else torch.int32
        assert torch.equal(x.view(bits), y.view(bits))


def host_state(state):
    return (helpers.tensor_to_numpy(state[0]), helpers.tensor_to_numpy(state[1]),
            [helpers.tensor_to_numpy(p) for p in state[2]])


# sizes: several tiles plus a ragged tail (the last level's tail is not a whole 16-byte unit),
# all levels 16-byte aligned / deliberately misaligned
ALIGNED = {3: (3 * 2048 + 72, 2 * 2048 + 8, 5 * 2048 + 1003),
           5: (3 * 2048 + 72, 2 * 2048 + 8, 2048 + 1000, 4096, 4096 + 21)}
ODD = {3: (50003, 50003, 50003), 5: (20003, 10001, 10001, 10001, 10001)}


@pytest.mark.parametrize("kernel", [B.DIPACO_KERNEL_AUTO, B.DIPACO_KERNEL_VECTOR, B.DIPACO_KERNEL_SCALAR])
def test_grid2x2_full_parity(kernel):
    pr = synth.make_problem(synth.CONFIGS["grid2x2"], DEV)
    before = host_state(clone_problem(pr))
    state = clone_problem(pr)
    run_gpu(pr, state, kernel=kernel)
    assert_matches_oracle(pr, before, state)


def test_grid4x4_full_parity_token_weights_and_momentum():
    pr = synth.make_problem(synth.CONFIGS["grid4x4"], DEV)
    before = host_state(clone_problem(pr))
    state = clone_problem(pr)
    run_gpu(pr, state)
    assert_matches_oracle(pr, before, state)


@pytest.mark.parametrize("name", ["grid16x16", "grid16x16-masked", "grid4x4x4x4"])
@pytest.mark.parametrize("sizes", ["aligned", "odd"])
def test_large_grids_scaled_full_parity(name, sizes):
    base = synth.CONFIGS[name]
    numel = (ALIGNED if sizes == "aligned" else ODD)[base.num_levels]
    pr = synth.make_problem(base.scaled(numel), DEV)
    before = host_state(clone_problem(pr))
    state = clone_problem(pr)
    run_gpu(pr, state)
    assert_matches_oracle(pr, before, state)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_kernel_families_and_tunings_agree_bitwise(dtype):
    cfg = synth.SyncConfig("mix", (1, 4, 4), (5 * 4096 + 24, 3 * 4096 + 8, 4096 * 2 + 120), dtype,
                           weights="tokens", momentum_std=1e-4, mask_prob=0.2, seed=5)
    pr = synth.make_problem(cfg, DEV)
    ref = clone_problem(pr)
    run_gpu(pr, ref, kernel=B.DIPACO_KERNEL_SCALAR)
    for kernel, tuning in [(B.DIPACO_KERNEL_VECTOR, None), (B.DIPACO_KERNEL_AUTO, None),
                           (B.DIPACO_KERNEL_AUTO, (1, 3, 1)), (B.DIPACO_KERNEL_AUTO, (1, 0, 2)),
                           (B.DIPACO_KERNEL_AUTO, (2, 2, 1)), (B.DIPACO_KERNEL_AUTO, (1, 0, 4)),
                           (B.DIPACO_KERNEL_AUTO, (3, 0, 1)), (B.DIPACO_KERNEL_AUTO, (1, 6, 2, 4)),
                           (B.DIPACO_KERNEL_AUTO, (1, 4, 1, 2))]:
        state = clone_problem(pr)
        run_gpu(pr, state, kernel=kernel, tuning=tuning)
        assert_states_bitwise_equal(ref, state)


@pytest.mark.parametrize("name", ["grid16x16", "grid16x16-masked", "grid4x4x4x4"])
def test_chunked_mode_is_bitwise_identical_to_resident(name):
    base = synth.CONFIGS[name]
    pr = synth.make_problem(base.scaled(ALIGNED[base.num_levels]), DEV)
    resident = clone_problem(pr)
    run_gpu(pr, resident, chunk_paths=0)
    for chunk in (32, 100):
        chunked = clone_problem(pr)
        launches = run_gpu(pr, chunked, chunk_paths=chunk)
        assert launches > 2
        assert_states_bitwise_equal(resident, chunked)


@pytest.mark.parametrize("kernel", [B.DIPACO_KERNEL_AUTO, B.DIPACO_KERNEL_VECTOR, B.DIPACO_KERNEL_SCALAR])
@pytest.mark.parametrize("empty_module", [False, True])
def test_incremental_api_with_fresh_buffers_for_writeback(kernel, empty_module):
    """The chunk API as a streaming caller uses it.  With bf16 copies the write-back launches read
    cast(theta') from the scratch that the finishing passes filled; a module that nobody updated
    has no entry there and is filled from theta."""
    base = synth.CONFIGS["grid16x16-masked"]
    pr = synth.make_problem(base.scaled(ALIGNED[3]), DEV)
    if empty_module:
        pr.reported = pr.reported.copy()
        pr.reported[[i for i in range(256) if pr.table[i, 2] == 9]] = 0
    resident = clone_problem(pr)
    run_gpu(pr, resident)
    theta, momentum, paths = clone_problem(pr)
    ctx = make_ctx(pr, chunk_paths=32, kernel=kernel)
    nchunks, scratch = B.dipaco_plan_chunks(ctx)
    assert nchunks == 8 and scratch > 0
    B.dipaco_sync_begin(ctx, theta.data_ptr(), momentum.data_ptr(), pr.reported)
    # out-of-order chunk is refused and changes nothing
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_sync_accumulate(ctx, 1, [p.data_ptr() for p in paths[32:64]])
    assert e.value.status == B.DIPACO_ESTATE
    with pytest.raises(B.DipacoError):
        B.dipaco_sync_writeback(ctx, 0, [p.data_ptr() for p in paths[0:32]])
    for c in range(nchunks):
        # each chunk is staged through the same device buffer, as a streaming caller would
        stage = [p.clone() for p in paths[32 * c:32 * c + 32]]
        B.dipaco_sync_accumulate(ctx, c, [p.data_ptr() for p in stage])
        torch.cuda.synchronize()
    out_paths = []
    for c in range(nchunks):
        fresh = [torch.full_like(p, float("nan")) for p in paths[32 * c:32 * c + 32]]
        B.dipaco_sync_writeback(ctx, c, [p.data_ptr() for p in fresh])
        out_paths.extend(fresh)
    B.dipaco_sync_end(ctx)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    assert_states_bitwise_equal((theta, momentum, out_paths), resident)


def test_forced_empty_module_and_all_masked_call():
    base = synth.CONFIGS["grid16x16-masked"]
    pr = synth.make_problem(base.scaled(ALIGNED[3]), DEV)
    reported = pr.reported.copy()
    reported[[i for i in range(256) if pr.table[i, 1] == 3]] = 0   # level-1 module 3 loses everyone
    for chunk in (0, 32):
        before = host_state(clone_problem(pr))
        state = clone_problem(pr)
        run_gpu(pr, state, reported=reported, chunk_paths=chunk)
        assert_matches_oracle(pr, before, state, reported=reported)
        n0, n1, _ = pr.cfg.level_numel
        sl = slice(n0 + 3 * n1, n0 + 4 * n1)
        assert torch.equal(state[0][sl].view(torch.int32), pr.theta[sl].view(torch.int32))
        assert torch.equal(state[1][sl].view(torch.int32), pr.momentum[sl].view(torch.int32))
    none = np.zeros(256, dtype=np.uint8)
    state = clone_problem(pr)
    run_gpu(pr, state, reported=none)
    assert torch.equal(state[0].view(torch.int32), pr.theta.view(torch.int32))
    assert torch.equal(state[1].view(torch.int32), pr.momentum.view(torch.int32))
    before = host_state(clone_problem(pr))
    assert_matches_oracle(pr, before, state, reported=none)


def test_masked_paths_are_not_read_and_nan_propagates():
    cfg = synth.CONFIGS["grid4x4"].scaled((4096 + 8, 2048 + 16, 2048))
    pr = synth.make_problem(cfg, DEV)
    reported = np.ones(16, dtype=np.uint8)
    reported[5] = 0
    clean = clone_problem(pr)
    run_gpu(pr, clean, reported=reported)
    dirty = clone_problem(pr)
    dirty[2][5].fill_(float("nan"))
    run_gpu(pr, dirty, reported=reported)
    assert_states_bitwise_equal(clean, dirty)
    # a NaN in a reporting copy reaches exactly the elements it touches
    state = clone_problem(pr)
    state[2][2][7] = float("nan")
    run_gpu(pr, state, reported=reported)
    assert torch.isnan(state[0][7]) and not torch.isnan(state[0][8])
    assert torch.isnan(state[0]).sum().item() == 1


def test_misaligned_path_pointers_on_small_modules():
    cfg = synth.SyncConfig("mis", (1, 2, 2), (4100, 2052, 1000), "bf16", seed=9)
    pr = synth.make_problem(cfg, DEV)
    before = host_state(clone_problem(pr))
    per = cfg.params_per_path
    backing = [torch.empty(per + 8, dtype=torch.bfloat16, device=DEV) for _ in range(4)]
    paths = []
    for i, b in enumerate(backing):
        view = b[1 + i:1 + i + per]          # 2-byte aligned only
        view.copy_(pr.paths[i])
        paths.append(view)
    state = (pr.theta.clone(), pr.momentum.clone(), paths)
    run_gpu(pr, state)
    assert_matches_oracle(pr, before, state)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("chunk", [0, 4])
def test_path_buffers_at_any_element_alignment(dtype, chunk):
    """Every path copy starts at its own element offset within a 16-byte unit (all eight of them
    for bf16, all four for fp32) and the level sizes are odd, so the modules of theta, the slots
    inside the copies and the partial sums all start inside 16-byte units.  The bulk-copy kernel
    (default) or the vector kernel, each in its variant for shifted buffers, takes the bulk of
    every module, the one-element kernel a few elements before and after: against the oracle,
    and bitwise equal to the one-element kernel on its own."""
    cfg = synth.SyncConfig("shifted", (1, 3, 3), (3 * 2048 + 5, 2 * 2048 + 1003, 5 * 2048 + 77), dtype,
                           weights="tokens", momentum_std=1e-4, seed=9)
    pr = synth.make_problem(cfg, DEV)
    before = host_state(clone_problem(pr))
    per = cfg.params_per_path
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    slots = 16 // (2 if dtype == "bf16" else 4)
    reported = np.ones(cfg.num_paths, dtype=np.uint8)
    reported[4] = 0

    def misaligned_state():
        backing = [torch.empty(per + 16, dtype=tdt, device=DEV) for _ in range(cfg.num_paths)]
        paths = []
        for i, b in enumerate(backing):
            off = i % slots
            view = b[off:off + per]
            view.copy_(pr.paths[i])
            assert view.data_ptr() % 16 == off * view.element_size()
            paths.append(view)
        return (pr.theta.clone(), pr.momentum.clone(), paths), backing

    results = {}
    for kernel in (B.DIPACO_KERNEL_AUTO, B.DIPACO_KERNEL_VECTOR, B.DIPACO_KERNEL_SCALAR):
        state, backing = misaligned_state()
        guard = [b.clone() for b in backing]
        launches = run_gpu(pr, state, reported=reported, chunk_paths=chunk, kernel=kernel)
        if chunk == 0:
            # one launch of the one-element kernel alone; with the vector kernel one more
            assert launches == (1 if kernel == B.DIPACO_KERNEL_SCALAR else 2)
        assert_matches_oracle(pr, before, state, reported=reported)
        # nothing outside the copies was written (the stores of aligned units stop at the edges)
        for i, (b, g) in enumerate(zip(backing, guard)):
            off = i % slots
            bits = torch.int16 if dtype == "bf16" else torch.int32
            assert torch.equal(b[:off].view(bits), g[:off].view(bits))
            assert torch.equal(b[off + per:].view(bits), g[off + per:].view(bits))
        results[kernel] = state
    assert_states_bitwise_equal(results[B.DIPACO_KERNEL_AUTO], results[B.DIPACO_KERNEL_SCALAR])
    assert_states_bitwise_equal(results[B.DIPACO_KERNEL_VECTOR], results[B.DIPACO_KERNEL_SCALAR])


def test_runs_are_bitwise_reproducible():
    base = synth.CONFIGS["grid4x4x4x4"]
    cfg = base.scaled((20 * 2048 + 8, 10 * 2048, 10 * 2048 + 16, 10 * 2048, 10 * 2048 + 1000))
    results = []
    for _ in range(3):
        pr = synth.make_problem(cfg, DEV)       # regenerated from the seed every time
        state = (pr.theta, pr.momentum, pr.paths)
        run_gpu(pr, state)
        results.append(state)
    assert_states_bitwise_equal(results[0], results[1])
    assert_states_bitwise_equal(results[0], results[2])


def test_two_rounds_on_one_context_follow_the_oracle():
    cfg = synth.CONFIGS["grid4x4"].scaled((3 * 2048 + 24, 2048 + 8, 2048 + 40))
    pr = synth.make_problem(cfg, DEV)
    th, mo, ps = host_state(clone_problem(pr))
    theta, momentum, paths = clone_problem(pr)
    ctx = make_ctx(pr)
    rng = np.random.RandomState(3)
    for rnd in range(2):
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths],
                            pr.reported)
        th, mo, ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, pr.weights, pr.reported)
        err = np.abs(helpers.tensor_to_numpy(theta).astype(np.float64) - th)
        assert np.all(err <= 1e-6 * (1 + np.abs(th)))
        # next inner phase: every path drifts away from the synchronised value again
        for i in range(cfg.num_paths):
            drift = rng.normal(0, 1e-3, cfg.params_per_path).astype(np.float32)
            ps[i] = ps[i] + drift
            paths[i].copy_(torch.from_numpy(ps[i]))
        # keep the oracle's global state equal to the device's so errors do not compound
        th = helpers.tensor_to_numpy(theta)
        mo = helpers.tensor_to_numpy(momentum)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    assert B.dipaco_launch_count(ctx) >= 2
    B.dipaco_destroy(ctx)


def test_argument_errors_leave_buffers_untouched():
    pr = synth.make_problem(synth.CONFIGS["grid2x2"], DEV)
    state = clone_problem(pr)
    ctx = make_ctx(pr)
    ptrs = [p.data_ptr() for p in state[2]]
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_outer_sync(ctx, 0, state[1].data_ptr(), ptrs)
    assert e.value.status == B.DIPACO_EINVAL
    with pytest.raises(B.DipacoError):
        B.dipaco_outer_sync(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs[:3] + [0])
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_sync_begin(ctx, state[0].data_ptr(), state[1].data_ptr())   # not a chunked context
    assert e.value.status == B.DIPACO_ESTATE
    torch.cuda.synchronize()
    assert_states_bitwise_equal(state, clone_problem(pr))
    B.dipaco_destroy(ctx)


@pytest.mark.parametrize("name,pinned", [("grid16x16-masked", True), ("grid4x4", False)])
def test_host_buffers_entry_point_matches_the_oracle(name, pinned):
    base = synth.CONFIGS[name]
    numel = ALIGNED[3] if name != "grid4x4" else (3 * 2048 + 24, 2048 + 8, 50003)
    cfg = base.scaled(numel)
    pr = synth.make_problem(cfg, "cpu")
    before = host_state(clone_problem(pr))
    theta, momentum, paths = clone_problem(pr)
    if pinned:
        theta, momentum = theta.pin_memory(), momentum.pin_memory()
        paths = [p.pin_memory() for p in paths]
    chunk = 32 if cfg.num_paths > 32 else 5
    ctx = make_ctx(pr, chunk_paths=chunk)
    # default: host threads fan each module's result out to its paths; then the same with three
    # threads and with none (one output row per path, all downloaded); later calls reuse the staging
    for rnd, threads in enumerate((-1, 3, 0)):
        B.dipaco_set_host_threads(ctx, threads)
        if rnd > 0:
            theta.copy_(pr.theta); momentum.copy_(pr.momentum)
            for p, q in zip(paths, pr.paths):
                p.copy_(q)
        B.dipaco_outer_sync_host(ctx, theta.data_ptr(), momentum.data_ptr(),
                                 [p.data_ptr() for p in paths], pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        assert_matches_oracle(pr, before, (theta, momentum, paths))
    B.dipaco_destroy(ctx)
    # and it is bitwise the device-resident result
    dev = synth.make_problem(cfg, "cpu")
    state = (dev.theta.to(DEV), dev.momentum.to(DEV), [p.to(DEV) for p in dev.paths])
    run_gpu(pr, state)
    assert_states_bitwise_equal((theta.to(DEV), momentum.to(DEV), [p.to(DEV) for p in paths]), state)


@pytest.mark.parametrize("mode", ["resident", "chunked", "host"])
def test_gradient_rescaling_and_levels_kept_local(mode):
    """Section 2.7 rescaling (here sqrt of the number of paths through each module) and a level
    that takes no part in the exchange, against the oracle, in every mode."""
    base = synth.CONFIGS["grid16x16-masked"]
    cfg = base.scaled((2 * 4096 + 72, 4096 + 8, 3 * 4096 + 1003))
    pr = synth.make_problem(cfg, "cpu" if mode == "host" else DEV)
    before = host_state(clone_problem(pr))
    scale = np.concatenate([[np.sqrt(256.0)], np.full(16, np.sqrt(16.0)),
                            np.sqrt(np.arange(1, 17))]).astype(np.float32)
    flags = np.array([1, 0, 1], dtype=np.uint8)
    theta, momentum, paths = clone_problem(pr)
    ctx = make_ctx(pr, chunk_paths=0 if mode == "resident" else 32)
    B.dipaco_set_module_scale(ctx, scale)
    B.dipaco_set_level_sync(ctx, flags)
    ptrs = [p.data_ptr() for p in paths]
    if mode == "host":
        B.dipaco_outer_sync_host(ctx, theta.data_ptr(), momentum.data_ptr(), ptrs, pr.reported)
    else:
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), ptrs, pr.reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    want_th, want_mo, want_ps = helpers.run_oracle(cfg, pr.table, *before, pr.weights, pr.reported,
                                                   num_threads=8, module_scale=scale.astype(np.float64),
                                                   level_sync=flags)
    got_th, got_mo = helpers.tensor_to_numpy(theta), helpers.tensor_to_numpy(momentum)
    for got, want in ((got_th, want_th), (got_mo, want_mo)):
        err = np.abs(got.astype(np.float64) - want.astype(np.float64))
        assert np.all(err <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
    n0, n1, n2 = cfg.level_numel
    # the level kept local is bitwise untouched everywhere
    np.testing.assert_array_equal(got_th[n0:n0 + 16 * n1], before[0][n0:n0 + 16 * n1])
    np.testing.assert_array_equal(got_mo[n0:n0 + 16 * n1], before[1][n0:n0 + 16 * n1])
    for i, p in enumerate(paths):
        got = helpers.tensor_to_numpy(p)
        np.testing.assert_array_equal(got[n0:n0 + n1], before[2][i][n0:n0 + n1])
        assert_bf16_close(got[:n0], want_ps[i][:n0])
        assert_bf16_close(got[n0 + n1:], want_ps[i][n0 + n1:])
    assert not np.array_equal(got_th[:n0], before[0][:n0])


def custom_problem(K, numel, table, dtype, seed, device=DEV, momentum_std=1e-4):
    """A problem on an arbitrary path table (not the full product of the levels)."""
    cfg = synth.SyncConfig("custom", tuple(K), tuple(numel), dtype, momentum_std=momentum_std, seed=seed)
    table = np.ascontiguousarray(table, dtype=np.int32)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    theta = torch.empty(cfg.module_params, device=device).normal_(0, 0.02, generator=gen)
    momentum = torch.empty(cfg.module_params, device=device).normal_(0, momentum_std, generator=gen)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    mod_off = np.concatenate([[0], np.cumsum([k * n for k, n in zip(K, numel)])])
    paths = []
    for i in range(table.shape[0]):
        parts = []
        for l, n in enumerate(numel):
            src = int(mod_off[l]) + int(table[i, l]) * n
            parts.append(theta[src:src + n] + torch.empty(n, device=device).normal_(0, 1e-3, generator=gen))
        paths.append(torch.cat(parts).to(tdt))
    return synth.SyncProblem(cfg, table, None, None, theta, momentum, paths)


@pytest.mark.parametrize("case", ["diloco", "flat", "sampled_paths", "empty_level", "tiny_modules",
                                  "many_paths"])
def test_special_structures_match_the_oracle(case):
    if case == "diloco":            # one level, one module, eight workers (Section 2.5)
        pr = custom_problem((1,), (3 * 4096 + 40,), np.zeros((8, 1)), "bf16", 1)
    elif case == "flat":            # no sharing at all: one level, K = P (Section 2.6.3)
        pr = custom_problem((64,), (4096 + 24,), np.arange(64).reshape(64, 1), "bf16", 2)
    elif case == "sampled_paths":   # three of the nine paths of a 3x3 grid; one module unused
        pr = custom_problem((1, 3, 3), (4104, 2056, 4096), [[0, 0, 1], [0, 2, 1], [0, 2, 2]], "f32", 3)
    elif case == "empty_level":     # a level without parameters
        pr = custom_problem((1, 2, 2), (4096, 0, 2048 + 8), synth.path_table((1, 2, 2)), "bf16", 4)
    elif case == "tiny_modules":    # modules smaller than one 16-byte unit
        pr = custom_problem((1, 2, 2), (3, 1, 5), synth.path_table((1, 2, 2)), "bf16", 5)
    else:                           # 1000 paths through one module, 125 modules of 8 paths
        table = np.stack([np.zeros(1000, np.int64), np.arange(1000) // 8], axis=1)
        pr = custom_problem((1, 125), (2 * 4096 + 16, 4096), table, "bf16", 6)
    for chunk in (0, 3):
        before = host_state(clone_problem(pr))
        state = clone_problem(pr)
        run_gpu(pr, state, chunk_paths=chunk)
        assert_matches_oracle(pr, before, state)
        if case == "sampled_paths":   # the module nobody passes through is never touched
            n0, n1 = pr.cfg.level_numel[0], pr.cfg.level_numel[1]
            sl = slice(n0 + n1, n0 + 2 * n1)
            assert torch.equal(state[0][sl], pr.theta[sl]) and torch.equal(state[1][sl], pr.momentum[sl])


@pytest.mark.parametrize("mode", ["resident", "chunked", "host"])
def test_shards_together_equal_the_unsharded_update(mode):
    """Three contexts, each owning one slab of every module, applied one after another to the same
    buffers, give bitwise the unsharded result; each touches only its own slabs."""
    base = synth.CONFIGS["grid4x4"]
    cfg = synth.SyncConfig("shards", (1, 4, 4), (5 * 8192 + 4096 + 24, 3 * 8192 + 8, 2 * 8192 + 1003),
                           "bf16", weights="tokens", momentum_std=1e-4, mask_prob=0.2, seed=11)
    dev = "cpu" if mode == "host" else DEV
    pr = synth.make_problem(cfg, dev)
    whole = clone_problem(pr)
    ctx = make_ctx(pr, chunk_paths=0 if mode == "resident" else 5)

    def call(state):
        ptrs = [p.data_ptr() for p in state[2]]
        fn = B.dipaco_outer_sync_host if mode == "host" else B.dipaco_outer_sync
        fn(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs, pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK

    call(whole)
    parts = clone_problem(pr)
    changed_so_far = torch.zeros_like(parts[0], dtype=torch.bool)
    for shard in range(3):
        B.dipaco_set_shard(ctx, shard, 3)
        before = parts[0].clone()
        call(parts)
        changed = parts[0] != before
        assert changed.any() and not (changed & changed_so_far).any()
        changed_so_far |= changed
    B.dipaco_set_shard(ctx, 0, 1)
    B.dipaco_destroy(ctx)
    assert_states_bitwise_equal(whole, parts)
    with pytest.raises(B.DipacoError):
        c2 = make_ctx(pr)
        try:
            B.dipaco_set_shard(c2, 3, 3)
        finally:
            B.dipaco_destroy(c2)


@pytest.mark.parametrize("opt", [B.DIPACO_OPT_MOMENTUM, B.DIPACO_OPT_SGD])
@pytest.mark.parametrize("chunk", [0, 32])
def test_other_outer_optimizers_match_the_oracle(opt, chunk):
    base = synth.CONFIGS["grid16x16-masked"]
    cfg = dataclass_replace(base.scaled((4096 + 72, 4096 + 8, 2 * 4096 + 1003)), momentum_std=1e-4)
    pr = synth.make_problem(cfg, DEV)
    before = host_state(clone_problem(pr))
    theta, momentum, paths = clone_problem(pr)
    ctx = make_ctx(pr, chunk_paths=chunk)
    B.dipaco_set_optimizer(ctx, opt)
    B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths],
                        pr.reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    want_th, want_mo, want_ps = helpers.run_oracle(cfg, pr.table, *before, pr.weights, pr.reported,
                                                   num_threads=8, optimizer=int(opt))
    for got, want in ((helpers.tensor_to_numpy(theta), want_th), (helpers.tensor_to_numpy(momentum), want_mo)):
        err = np.abs(got.astype(np.float64) - want.astype(np.float64))
        assert np.all(err <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
    if opt == B.DIPACO_OPT_SGD:
        assert torch.equal(momentum.view(torch.int32), pr.momentum.view(torch.int32))
    for i in range(0, cfg.num_paths, 7):
        assert_bf16_close(helpers.tensor_to_numpy(paths[i]), want_ps[i])


def dataclass_replace(cfg, **kw):
    import dataclasses
    return dataclasses.replace(cfg, **kw)


def test_calls_run_on_the_callers_stream():
    """Work is ordered on the stream that is passed in: producer and consumer kernels queued on a
    side stream around the call see consistent data without any device-wide synchronisation."""
    cfg = synth.CONFIGS["grid4x4"].scaled((6 * 4096 + 8, 4096 + 16, 2 * 4096))
    pr = synth.make_problem(cfg, DEV)
    ref = clone_problem(pr)
    run_gpu(pr, ref)
    side = torch.cuda.Stream()
    theta, momentum, paths = clone_problem(pr)
    torch.cuda.synchronize()
    ctx = make_ctx(pr)
    with torch.cuda.stream(side):
        # inputs are produced on the side stream right before the call ...
        staged = [p.clone() for p in paths]
        for p in paths:
            p.zero_()
        for p, q in zip(paths, staged):
            p.copy_(q)
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths],
                            pr.reported, stream=side)
        # ... and consumed on it right after
        total = sum(float(p.double().sum()) for p in paths[:2])
    side.synchronize()
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)
    want = sum(float(p.double().sum()) for p in ref[2][:2])
    assert abs(total - want) <= 1e-4 * (1 + abs(want))
    err = (theta.double() - ref[0].double()).abs()
    assert bool((err <= 1e-6 * (1 + ref[0].double().abs())).all())


@pytest.mark.parametrize("variant", ["federated", "adamw_gradients"])
@pytest.mark.parametrize("chunk,kernel", [(0, B.DIPACO_KERNEL_AUTO), (32, B.DIPACO_KERNEL_AUTO),
                                          (0, B.DIPACO_KERNEL_VECTOR), (5, B.DIPACO_KERNEL_SCALAR)])
def test_adam_family_and_gradient_inputs_match_the_oracle(variant, chunk, kernel):
    base = synth.CONFIGS["grid16x16-masked"]
    cfg = dataclass_replace(base.scaled((4096 + 72, 2 * 4096 + 8, 4096 + 1003)), momentum_std=1e-4)
    pr = synth.make_problem(cfg, DEV)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(3)
    second = torch.empty_like(pr.theta).normal_(0, 1e-4, generator=gen).abs_()
    if variant == "adamw_gradients":
        # the buffers hold gradients, not copies; two consecutive steps of bias-corrected AdamW
        for p in pr.paths:
            p.copy_(torch.empty(p.numel(), device=DEV).normal_(0, 1e-2, generator=gen))
        lr, adam_args, steps, kind = 4e-4, (0.9, 0.999, 1e-8, 0.1), (1, 2), B.DIPACO_INPUT_GRADIENTS
    else:
        lr, adam_args, steps, kind = 0.1, (0.9, 0.99, 1e-3, 0.0), (0,), B.DIPACO_INPUT_COPIES
    theta, momentum, paths = clone_problem(pr)
    v = second.clone()
    th, mo, ps = host_state((theta, momentum, paths))
    v_host = helpers.tensor_to_numpy(v)
    code = B.DIPACO_BF16
    ctx = B.dipaco_create(cfg.modules_per_level, cfg.level_numel, pr.table, pr.weights, np.float32(lr),
                          np.float32(0.9), code, chunk, 0)
    B.dipaco_set_kernel(ctx, kernel)
    B.dipaco_set_input_kind(ctx, kind)
    for step in steps:
        B.dipaco_set_adam(ctx, v.data_ptr(), *adam_args, step)
        B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths],
                            pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        b1, b2, eps, wd = [float(np.float32(x)) for x in adam_args]
        c1 = 1 - b1 ** step if step else 1.0
        c2 = 1 - b2 ** step if step else 1.0
        th, mo, ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, pr.weights, pr.reported, lr=lr,
                                        num_threads=8, optimizer=3, second_moment=v_host,
                                        adam=(b1, b2, eps, wd, c1, c2), input_kind=int(kind))
        for got, want in ((theta, th), (momentum, mo), (v, v_host)):
            g = helpers.tensor_to_numpy(got).astype(np.float64)
            assert np.all(np.abs(g - want) <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
        for i in range(0, cfg.num_paths, 9):
            assert_bf16_close(helpers.tensor_to_numpy(paths[i]), ps[i])
        if len(steps) > 1:
            # next step: fresh gradients in the buffers, oracle continues from the device state
            th, mo = helpers.tensor_to_numpy(theta), helpers.tensor_to_numpy(momentum)
            v_host = helpers.tensor_to_numpy(v)
            for i, p in enumerate(paths):
                p.copy_(torch.empty(p.numel(), device=DEV).normal_(0, 1e-2, generator=gen))
                ps[i] = helpers.tensor_to_numpy(p)
    B.dipaco_destroy(ctx)


def test_adam_needs_its_second_moment_first():
    pr = synth.make_problem(synth.CONFIGS["grid2x2"], DEV)
    ctx = make_ctx(pr)
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_set_optimizer(ctx, B.DIPACO_OPT_ADAM)
    assert e.value.status == B.DIPACO_ESTATE
    with pytest.raises(B.DipacoError):
        B.dipaco_set_adam(ctx, pr.theta.data_ptr(), 1.0, 0.9, 1e-8, 0.0, 0)
    B.dipaco_destroy(ctx)


def test_adam_family_through_the_host_buffer_entry_point():
    """theta, momentum, the second moment and the path copies all live in host memory; the result
    is bitwise the device-resident one."""
    base = synth.CONFIGS["grid16x16-masked"]
    cfg = dataclass_replace(base.scaled((4096 + 72, 2 * 4096 + 8, 4096 + 1003)), momentum_std=1e-4)
    pr = synth.make_problem(cfg, "cpu")
    second = torch.empty_like(pr.theta).normal_(0, 1e-4).abs_()
    host = [t.clone().pin_memory() for t in (pr.theta, pr.momentum, second)]
    host_paths = [p.clone().pin_memory() for p in pr.paths]
    dev = [t.to(DEV) for t in (pr.theta, pr.momentum, second)]
    dev_paths = [p.to(DEV) for p in pr.paths]
    for where, (theta, momentum, v), paths in (("host", host, host_paths), ("device", dev, dev_paths)):
        ctx = make_ctx(pr, chunk_paths=32 if where == "host" else 0)
        B.dipaco_set_adam(ctx, v.data_ptr(), 0.9, 0.99, 1e-3, 0.01, 3)
        fn = B.dipaco_outer_sync_host if where == "host" else B.dipaco_outer_sync
        fn(ctx, theta.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in paths], pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        B.dipaco_destroy(ctx)
    for a, b in zip(host, dev):
        assert torch.equal(a.view(torch.int32), b.cpu().view(torch.int32))
    for a, b in zip(host_paths, dev_paths):
        assert torch.equal(a.view(torch.int16), b.cpu().view(torch.int16))
    assert not torch.equal(host[2], second)


def test_a_repeated_call_reuses_its_plan_and_any_change_replans():
    """dipaco_outer_sync keeps the plan of the previous call while settings, buffers and mask stay
    the same; whatever changes (mask, weights, a path buffer, theta) must give the result of a
    fresh context."""
    cfg = synth.CONFIGS["grid4x4"].scaled((3 * 4096 + 24, 4096 + 8, 2 * 4096 + 1003))
    pr = synth.make_problem(cfg, DEV)

    def fresh(reported, weights, order=None):
        state = clone_problem(pr)
        if order is not None:
            state = (state[0], state[1], [state[2][i] for i in order])
        run_gpu(pr, state, reported=reported, weights=weights)
        return state

    ctx = make_ctx(pr)
    theta, momentum, paths = clone_problem(pr)

    def restore():
        theta.copy_(pr.theta); momentum.copy_(pr.momentum)
        for p, q in zip(paths, pr.paths):
            p.copy_(q)

    def call(reported, bufs=None, th=None):
        bufs = paths if bufs is None else bufs
        th = theta if th is None else th
        B.dipaco_outer_sync(ctx, th.data_ptr(), momentum.data_ptr(), [p.data_ptr() for p in bufs], reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK

    for _ in range(3):                       # identical calls: the second and third reuse the plan
        restore()
        call(pr.reported)
        assert_states_bitwise_equal((theta, momentum, paths), fresh(pr.reported, pr.weights))
    mask = np.ones(16, dtype=np.uint8)
    mask[[2, 11]] = 0
    restore(); call(mask)                    # another mask
    assert_states_bitwise_equal((theta, momentum, paths), fresh(mask, pr.weights))
    restore(); call(None)                    # no mask
    assert_states_bitwise_equal((theta, momentum, paths), fresh(None, pr.weights))
    w2 = pr.weights[::-1].copy()
    B.dipaco_set_weights(ctx, w2)            # other weights, same buffers and mask
    restore(); call(None)
    assert_states_bitwise_equal((theta, momentum, paths), fresh(None, w2))
    restore()                                # same set of buffers bound to other paths
    order = [1, 0] + list(range(2, 16))
    swapped = [paths[i] for i in order]
    for p, q in zip(swapped, pr.paths):
        p.copy_(q)
    call(None, bufs=swapped)
    want = fresh(None, w2)
    assert_states_bitwise_equal((theta, momentum, swapped), want)
    other_theta = pr.theta.clone()           # another theta buffer
    restore(); call(None, th=other_theta)
    assert_states_bitwise_equal((other_theta, momentum, paths), fresh(None, w2))
    B.dipaco_destroy(ctx)


@pytest.mark.parametrize("chunk", [0, 32])
def test_a_repeated_call_replayed_from_a_cuda_graph_follows_the_oracle(chunk):
    """A call that reuses the plan of the previous one only launches kernels (no upload, no
    allocation, no synchronisation), so it can be captured in a CUDA graph.  One replay on the
    original inputs matches the oracle; three replays give bitwise the result of three calls
    launched directly.  The ragged last level also puts the tail kernel in the graph."""
    cfg = synth.CONFIGS["grid16x16-masked"].scaled((2 * 4096 + 72, 4096 + 8, 4096 + 1003))
    pr = synth.make_problem(cfg, DEV)
    before = host_state(clone_problem(pr))
    direct = clone_problem(pr)
    ctx = make_ctx(pr, chunk)
    for _ in range(3):
        B.dipaco_outer_sync(ctx, direct[0].data_ptr(), direct[1].data_ptr(),
                            [p.data_ptr() for p in direct[2]], pr.reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)

    state = clone_problem(pr)
    ptrs = B.ptr_array([p.data_ptr() for p in state[2]])
    ctx = make_ctx(pr, chunk)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    # the call that plans and uploads the tables stays outside the graph
    B.dipaco_outer_sync(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs, pr.reported, stream=stream)
    stream.synchronize()
    launches_planned = B.dipaco_launch_count(ctx)
    assert launches_planned >= 2
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        B.dipaco_outer_sync(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs, pr.reported,
                            stream=torch.cuda.current_stream())
    assert B.dipaco_launch_count(ctx) == 2 * launches_planned

    def restore():
        state[0].copy_(pr.theta); state[1].copy_(pr.momentum)
        for p, q in zip(state[2], pr.paths):
            p.copy_(q)
        torch.cuda.synchronize()

    restore()
    graph.replay()
    torch.cuda.synchronize()
    assert_matches_oracle(pr, before, state)
    restore()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert_states_bitwise_equal(state, direct)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)


def test_a_wait_that_runs_out_is_reported_once_and_the_context_recovers():
    """The time-out path end to end, without disturbing the pipeline kernels: the diagnostic
    entry point makes one bounded wait (1 ms) run out on a barrier nothing completes.  The kernel
    must end by itself, later launches must do nothing while the error is pending,
    dipaco_device_status must report DIPACO_ETIMEOUT exactly once and re-arm the work counters,
    and the next synchronisation must be bitwise correct."""
    cfg = synth.CONFIGS["grid4x4"].scaled((6 * 4096 + 8, 4096 + 16, 2 * 4096 + 5))
    pr = synth.make_problem(cfg, DEV)
    ref = clone_problem(pr)
    run_gpu(pr, ref)
    for chunk in (0, 5):
        ctx = make_ctx(pr, chunk_paths=chunk)
        state = clone_problem(pr)
        ptrs = [p.data_ptr() for p in state[2]]
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        B.dipaco_selftest_wait_expiry(ctx, 1_000_000)
        end.record()
        torch.cuda.synchronize()
        ms = start.elapsed_time(end)
        assert 0.9 <= ms < 100.0, "the wait should give up after about 1 ms, took %.3f ms" % ms
        # the error is pending: this launch must leave everything as it is
        B.dipaco_outer_sync(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs, pr.reported)
        torch.cuda.synchronize()
        assert_states_bitwise_equal(state, clone_problem(pr))
        assert B.dipaco_device_status(ctx) == B.DIPACO_ETIMEOUT
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        # re-armed: the same call now does its work, and the work counters started from zero
        B.dipaco_outer_sync(ctx, state[0].data_ptr(), state[1].data_ptr(), ptrs, pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        assert_states_bitwise_equal(state, ref)
        with pytest.raises(B.DipacoError):
            B.dipaco_selftest_wait_expiry(ctx, 0)
        B.dipaco_destroy(ctx)


@pytest.mark.parametrize("mode", ["resident", "chunked", "host"])
def test_compact_shards_match_the_oracle_and_the_unsharded_update(mode):
    """Section 3.3, sharded executor: three executors that each hold ONLY their slab of theta,
    momentum and of every path copy (separate allocations, packed) update it through their own
    shard context; the slabs put back side by side equal the oracle's result for the whole
    problem and, bit for bit, the unsharded call."""
    cfg = synth.SyncConfig("shards", (1, 4, 4), (5 * 8192 + 4096 + 24, 3 * 8192 + 8, 2 * 8192 + 1003),
                           "bf16", weights="tokens", momentum_std=1e-4, mask_prob=0.2, seed=11)
    pr = synth.make_problem(cfg, DEV)
    before = host_state(clone_problem(pr))
    unsharded = clone_problem(pr)
    run_gpu(pr, unsharded)
    whole = make_ctx(pr, chunk_paths=0 if mode == "resident" else 5)
    B.dipaco_device_status(whole)
    S, L = 3, cfg.num_levels
    lvl, mod = pr.level_offsets(), pr.module_offsets()
    out = clone_problem(pr)
    where = "cpu" if mode == "host" else DEV

    def module_slices(bounds):
        for l, k in enumerate(cfg.modules_per_level):
            for e in range(k):
                base = int(mod[l]) + e * cfg.level_numel[l]
                yield slice(base + bounds[l][0], base + bounds[l][1])

    def path_slices(bounds):
        for l in range(L):
            yield slice(int(lvl[l]) + bounds[l][0], int(lvl[l]) + bounds[l][1])

    for s_idx in range(S):
        bounds = [B.dipaco_plan_shard(whole, s_idx, S, l) for l in range(L)]
        theta_s = torch.cat([pr.theta[sl] for sl in module_slices(bounds)]).to(where)
        mom_s = torch.cat([pr.momentum[sl] for sl in module_slices(bounds)]).to(where)
        paths_s = [torch.cat([p[sl] for sl in path_slices(bounds)]).to(where) for p in pr.paths]
        if mode == "host":
            theta_s, mom_s = theta_s.pin_memory(), mom_s.pin_memory()
            paths_s = [p.pin_memory() for p in paths_s]
        ctx = B.dipaco_create_shard(whole, s_idx, S, 0)
        fn = B.dipaco_outer_sync_host if mode == "host" else B.dipaco_outer_sync
        fn(ctx, theta_s.data_ptr(), mom_s.data_ptr(), [p.data_ptr() for p in paths_s], pr.reported)
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        B.dipaco_destroy(ctx)
        pos = 0
        for sl in module_slices(bounds):
            n = sl.stop - sl.start
            out[0][sl] = theta_s[pos:pos + n].to(DEV)
            out[1][sl] = mom_s[pos:pos + n].to(DEV)
            pos += n
        for i, p in enumerate(paths_s):
            pos = 0
            for sl in path_slices(bounds):
                n = sl.stop - sl.start
                out[2][i][sl] = p[pos:pos + n].to(DEV)
                pos += n
    B.dipaco_destroy(whole)
    assert_states_bitwise_equal(out, unsharded)
    assert_matches_oracle(pr, before, out)


def test_two_contexts_on_two_streams_do_not_disturb_each_other():
    """Contexts share nothing (tables, counters, error word and scratch are per context): two
    synchronisations queued back to back on different streams, so that they overlap on the
    device, each give bitwise their own result."""
    cfgs = [synth.CONFIGS["grid4x4"].scaled((24 * 4096 + 8, 8 * 4096 + 16, 8 * 4096)),
            synth.CONFIGS["grid16x16-masked"].scaled((4 * 4096 + 72, 2 * 4096 + 8, 4096 + 1003))]
    problems = [synth.make_problem(c, DEV) for c in cfgs]
    refs = []
    for pr, chunk in zip(problems, (0, 32)):
        ref = clone_problem(pr)
        run_gpu(pr, ref, chunk_paths=chunk)
        refs.append(ref)
    states = [clone_problem(pr) for pr in problems]
    ctxs = [make_ctx(problems[0], 0), make_ctx(problems[1], 32)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):
        for pr, st, ctx, stream in zip(problems, states, ctxs, streams):
            B.dipaco_outer_sync(ctx, st[0].data_ptr(), st[1].data_ptr(), [p.data_ptr() for p in st[2]],
                                pr.reported, stream=stream)
        for stream in streams:
            stream.synchronize()
        for pr, st, ref in zip(problems, states, refs):
            assert_states_bitwise_equal(st, ref)
            st[0].copy_(pr.theta); st[1].copy_(pr.momentum)      # restore for the next repetition
            for p, q in zip(st[2], pr.paths):
                p.copy_(q)
        torch.cuda.synchronize()
    for ctx in ctxs:
        assert B.dipaco_device_status(ctx) == B.DIPACO_OK
        B.dipaco_destroy(ctx)
