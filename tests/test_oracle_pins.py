"""Pins for the CPU oracle: closed forms, a library optimiser step, exact rational brute force.

Every check here compares the oracle with something that does not come from the oracle: a
closed form of the mathematics, numpy/torch library routines, or an exact-arithmetic restatement
of Algorithm 1's outer loop evaluated with Python fractions on tiny grids whose contributor sets
are the ones the paper states for its 2x2 figure (tests/golden/toy_2x2_contributors.txt).
"""
from __future__ import annotations

import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2403_10616_b200 import synth
from tests import helpers

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LR = float(np.float32(0.7))
MU = float(np.float32(0.9))


def tiny_cfg(K, numel, dtype="f32", **kw):
    return synth.SyncConfig("tiny", tuple(K), tuple(numel), dtype, **kw)


def one_ulp(x):
    return np.spacing(np.abs(np.asarray(x, dtype=np.float32)))


def module_slices(cfg):
    """[(level, module, theta slice, path slice)]"""
    out = []
    base = 0
    lvl = 0
    for l, (k, n) in enumerate(zip(cfg.modules_per_level, cfg.level_numel)):
        for e in range(k):
            out.append((l, e, slice(base, base + n), slice(lvl, lvl + n)))
            base += n
        lvl += n
    return out


def read_toy_sets():
    sets = {}
    with open(os.path.join(GOLDEN, "toy_2x2_contributors.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            left, right = line.split(":")
            lvl, mod = left.split()
            sets[(int(lvl) - 1, "ab".index(mod))] = [int(p) - 1 for p in right.split()]
    return sets


# ---------------------------------------------------------------------------- structure

def test_path_table_matches_the_papers_toy_figure():
    """Row-major path ids reproduce the sharing pattern the paper describes for the 2x2 toy."""
    table = synth.path_table((1, 2, 2))
    sets = read_toy_sets()
    for (l, e), want in sets.items():
        got = [i for i in range(4) if table[i, l] == e]
        assert got == want


def exact_reference(cfg, table, theta, momentum, paths, weights, reported, lr, mu, sets=None):
    """Algorithm 1's outer loop in exact rational arithmetic (inputs are binary floats, hence
    exact rationals).  `sets` optionally supplies the contributor sets instead of the table."""
    lr = Fraction(float(lr))
    mu = Fraction(float(mu))
    th_out = [Fraction(float(v)) for v in theta]
    mo_out = [Fraction(float(v)) for v in momentum]
    P = table.shape[0]
    for (l, e, ts, ps) in module_slices(cfg):
        S = sets[(l, e)] if sets is not None else [i for i in range(P) if table[i, l] == e]
        R = [i for i in S if reported is None or reported[i]]
        w = {i: Fraction(float(weights[i])) if weights is not None else Fraction(1) for i in R}
        W = sum(w.values(), Fraction(0))
        if not R or W == 0:
            continue
        for k in range(ts.stop - ts.start):
            t0 = Fraction(float(theta[ts.start + k]))
            delta = sum((w[i] / W) * (t0 - Fraction(float(paths[i][ps.start + k]))) for i in R)
            m1 = mu * Fraction(float(momentum[ts.start + k])) + delta
            th_out[ts.start + k] = t0 - lr * (delta + mu * m1)
            mo_out[ts.start + k] = m1
    return th_out, mo_out


def assert_close_to_exact(got, exact):
    exact_f = np.array([float(v) for v in exact], dtype=np.float64)
    err = np.abs(got.astype(np.float64) - exact_f)
    assert np.all(err <= one_ulp(exact_f.astype(np.float32)) * 0.5000001 + 1e-45), err.max()


def test_brute_force_exact_on_the_toy_2x2_with_the_papers_sets():
    cfg = tiny_cfg((1, 2, 2), (5, 7, 3), momentum_std=1e-2)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    ex_th, ex_mo = exact_reference(cfg, pr.table, th, mo, ps, None, None,
                                   np.float32(0.7), np.float32(0.9), sets=read_toy_sets())
    assert_close_to_exact(got_th, ex_th)
    assert_close_to_exact(got_mo, ex_mo)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_brute_force_exact_three_levels_weights_and_mask(dtype):
    cfg = tiny_cfg((2, 3, 2), (4, 3, 6), dtype, momentum_std=1e-2, seed=3)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    rng = np.random.RandomState(5)
    weights = rng.randint(1, 50, size=cfg.num_paths).astype(np.float32)
    reported = (rng.random_sample(cfg.num_paths) > 0.3).astype(np.uint8)
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, weights, reported)
    vals = [helpers.path_values(cfg, p) for p in ps]
    ex_th, ex_mo = exact_reference(cfg, pr.table, th, mo, vals, weights, reported,
                                   np.float32(0.7), np.float32(0.9))
    assert_close_to_exact(got_th, ex_th)
    assert_close_to_exact(got_mo, ex_mo)


# ---------------------------------------------------------------------------- closed forms

def dyadic(rng, n, scale):
    """Random values with few mantissa bits so sums and differences are exact in float."""
    return (rng.randint(-512, 513, size=n) * scale).astype(np.float32)


@pytest.mark.parametrize("weighted,masked", [(False, False), (True, False), (True, True)])
def test_identical_deltas_give_that_delta(weighted, masked):
    """All contributors hold theta - delta  =>  Delta = delta; from m = 0 the momentum becomes
    delta exactly and theta' = theta - lr*(1+mu)*delta."""
    cfg = tiny_cfg((1, 3, 2), (8, 5, 9))
    table = synth.path_table(cfg.modules_per_level)
    rng = np.random.RandomState(1)
    theta = dyadic(rng, cfg.module_params, 2.0 ** -12)
    delta = dyadic(rng, cfg.module_params, 2.0 ** -16)
    momentum = np.zeros_like(theta)
    paths = []
    for i in range(cfg.num_paths):
        row = np.empty(cfg.params_per_path, dtype=np.float32)
        for (l, e, ts, ps) in module_slices(cfg):
            if table[i, l] == e:
                row[ps] = theta[ts] - delta[ts]
        paths.append(row)
    weights = np.array([1, 2, 4, 8, 1, 2], dtype=np.float32) if weighted else None
    reported = np.array([1, 0, 1, 1, 1, 1], dtype=np.uint8) if masked else None
    th, mo, ps_out = helpers.run_oracle(cfg, table, theta, momentum, paths, weights, reported)
    # sum_i (w_i/W) * delta differs from delta only by double rounding of the w_i/W
    np.testing.assert_allclose(mo, delta, rtol=1e-7, atol=0)
    want = theta.astype(np.float64) - LR * (1.0 + MU) * delta.astype(np.float64)
    assert np.all(np.abs(th - want) <= one_ulp(want))


def test_lr_one_no_momentum_is_the_weighted_mean_of_copies():
    cfg = tiny_cfg((1, 2, 3), (16, 11, 7), momentum_std=1e-2, seed=4)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    rng = np.random.RandomState(9)
    weights = rng.randint(1000, 10001, size=cfg.num_paths).astype(np.float32)
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, weights, None,
                                               lr=1.0, mu=0.0)
    for (l, e, ts, psl) in module_slices(cfg):
        S = [i for i in range(cfg.num_paths) if pr.table[i, l] == e]
        stack = np.stack([ps[i][psl].astype(np.float64) for i in S])
        want = np.average(stack, axis=0, weights=weights[S].astype(np.float64))
        assert np.all(np.abs(got_th[ts] - want) <= one_ulp(want))


def test_unweighted_lr_one_is_the_plain_mean_and_masked_paths_are_excluded():
    cfg = tiny_cfg((1, 4), (6, 10), seed=8)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    reported = np.array([1, 1, 0, 1], dtype=np.uint8)
    got_th, _, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, None, reported, lr=1.0, mu=0.0)
    want_shared = np.mean(np.stack([ps[i][:6].astype(np.float64) for i in (0, 1, 3)]), axis=0)
    assert np.all(np.abs(got_th[:6] - want_shared) <= one_ulp(want_shared))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_single_path_returns_its_own_copy(dtype):
    cfg = tiny_cfg((1, 1), (9, 14), dtype, seed=2)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, lr=1.0, mu=0.0)
    np.testing.assert_array_equal(got_th, helpers.path_values(cfg, ps[0]))
    np.testing.assert_array_equal(got_ps[0], ps[0])
    np.testing.assert_array_equal(got_mo, th - helpers.path_values(cfg, ps[0]))


def test_module_without_reporting_path_is_left_unchanged():
    cfg = tiny_cfg((1, 2, 2), (4, 6, 5), "bf16", momentum_std=1e-2, seed=6)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    reported = np.array([0, 0, 1, 1], dtype=np.uint8)      # level-2 module 0 = paths {0, 1}
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, None, reported)
    sl = slice(4, 10)
    np.testing.assert_array_equal(got_th[sl].view(np.uint32), th[sl].view(np.uint32))
    np.testing.assert_array_equal(got_mo[sl].view(np.uint32), mo[sl].view(np.uint32))
    assert not np.array_equal(got_th[10:16], th[10:16])
    # its copies are still reset to the (unchanged) global value
    for i in (0, 1):
        np.testing.assert_array_equal(got_ps[i][4:10], helpers.float_to_bf16_bits_torch(th[sl]))
    # all paths masked: nothing moves at all
    none = np.zeros(4, dtype=np.uint8)
    got_th, got_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, None, none)
    np.testing.assert_array_equal(got_th.view(np.uint32), th.view(np.uint32))
    np.testing.assert_array_equal(got_mo.view(np.uint32), mo.view(np.uint32))
    # zero total weight counts as nobody reporting
    zero_w = np.array([0, 0, 1, 1], dtype=np.float32)
    got_th, got_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, zero_w, None)
    np.testing.assert_array_equal(got_th[sl].view(np.uint32), th[sl].view(np.uint32))


def test_constant_outer_gradient_follows_the_geometric_series():
    """Rounds with the same outer gradient g=1: momentum and step sizes of the golden file."""
    rows = []
    with open(os.path.join(GOLDEN, "nesterov_constant_gradient.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                t, m, s = line.split()
                rows.append((int(t), float(m), float(s)))
    cfg = tiny_cfg((1,), (3,))
    table = synth.path_table(cfg.modules_per_level)
    theta = np.array([10.0, -3.0, 0.5], dtype=np.float32)
    momentum = np.zeros(3, dtype=np.float32)
    for (t, want_m, want_step) in rows:
        paths = [theta - np.float32(1.0)]
        new_th, momentum, _ = helpers.run_oracle(cfg, table, theta, momentum, paths)
        np.testing.assert_allclose(momentum, want_m, rtol=3e-7)
        np.testing.assert_allclose(theta - new_th, want_step, rtol=0, atol=4e-6)
        theta = new_th


def test_zero_gradient_only_decays_momentum():
    cfg = tiny_cfg((1,), (4,))
    table = synth.path_table(cfg.modules_per_level)
    theta = np.array([1.0, 2.0, -1.0, 0.25], dtype=np.float32)
    momentum = np.array([0.5, -0.25, 1.0, 0.0], dtype=np.float32)
    th, mo, _ = helpers.run_oracle(cfg, table, theta, momentum, [theta.copy()])
    np.testing.assert_allclose(mo, MU * momentum.astype(np.float64), rtol=1e-7)
    np.testing.assert_allclose(th, theta - LR * MU * MU * momentum.astype(np.float64), rtol=2e-7)


def test_matches_torch_sgd_with_nesterov_momentum():
    """One library Nesterov step with .grad = Delta (Delta from numpy's mean)."""
    cfg = synth.SyncConfig("dense", (1,), (257,), "f32", momentum_std=1e-2, seed=11)
    table = np.zeros((5, 1), dtype=np.int32)            # five workers, one shared module
    pr = synth.make_problem(cfg)
    th, mo, _ = helpers.host_copy(pr)
    rng = np.random.RandomState(0)
    paths = [(th + rng.normal(0, 1e-3, size=257)).astype(np.float32) for _ in range(5)]
    # first round from zero momentum, second round carries the buffer
    param = torch.nn.Parameter(torch.from_numpy(th.copy()).double())
    opt = torch.optim.SGD([param], lr=LR, momentum=MU, nesterov=True)
    theta = th.copy()
    momentum = np.zeros_like(th)
    for rnd in range(2):
        delta = np.mean(np.stack([theta.astype(np.float64) - p.astype(np.float64) for p in paths]),
                        axis=0)
        param.grad = torch.from_numpy(delta.copy())
        with torch.no_grad():
            param.copy_(torch.from_numpy(theta.astype(np.float64)))
        opt.step()
        got_th, got_mo, got_ps = oracle_call(cfg, table, theta, momentum, paths)
        want = param.detach().numpy()
        assert np.all(np.abs(got_th - want) <= one_ulp(want))
        theta, momentum = got_th, got_mo
        paths = [(theta + rng.normal(0, 1e-3, size=257)).astype(np.float32) for _ in range(5)]


def oracle_call(cfg, table, theta, momentum, paths, **kw):
    th = theta.copy()
    mo = momentum.copy()
    ps = [p.copy() for p in paths]
    oracle.outer_sync(cfg.modules_per_level, cfg.level_numel, table, th, mo, ps, oracle.F32,
                      LR, MU, kw.get("weights"), kw.get("reported"))
    return th, mo, ps


def test_doubling_every_delta_doubles_the_outer_gradient():
    cfg = tiny_cfg((1, 2), (12, 20))
    table = synth.path_table(cfg.modules_per_level)
    rng = np.random.RandomState(12)
    theta = dyadic(rng, cfg.module_params, 2.0 ** -12)
    momentum = np.zeros_like(theta)

    def copies(scale):
        out = []
        for i in range(cfg.num_paths):
            row = np.empty(cfg.params_per_path, dtype=np.float32)
            r = np.random.RandomState(100 + i)
            row[:12] = theta[:12] - scale * dyadic(r, 12, 2.0 ** -16)
            e = table[i, 1]
            row[12:] = theta[12 + 20 * e:32 + 20 * e] - scale * dyadic(r, 20, 2.0 ** -16)
            out.append(row)
        return out

    _, mo1, _ = helpers.run_oracle(cfg, table, theta, momentum, copies(1))
    _, mo2, _ = helpers.run_oracle(cfg, table, theta, momentum, copies(2))
    assert np.any(mo1 != 0)
    np.testing.assert_array_equal(mo2, 2 * mo1)


# ---------------------------------------------------------------------------- special cases

def test_one_level_one_module_is_diloco_over_all_workers():
    cfg = synth.SyncConfig("diloco", (1,), (33,), "f32", seed=13)
    table = np.zeros((8, 1), dtype=np.int32)
    rng = np.random.RandomState(3)
    theta = rng.normal(0, 0.02, 33).astype(np.float32)
    momentum = rng.normal(0, 1e-2, 33).astype(np.float32)
    paths = [(theta + rng.normal(0, 1e-3, 33)).astype(np.float32) for _ in range(8)]
    th, mo, ps = oracle_call(cfg, table, theta, momentum, paths)
    delta = theta.astype(np.float64) - np.mean(np.stack(paths).astype(np.float64), axis=0)
    m1 = MU * momentum.astype(np.float64) + delta
    want = theta.astype(np.float64) - LR * (delta + MU * m1)
    assert np.all(np.abs(th - want) <= one_ulp(want))
    assert np.all(np.abs(mo - m1) <= one_ulp(m1))


def test_path_specific_modules_still_get_the_outer_optimizer():
    """Flat mixture: one level, K = P; each module is updated from its own path alone."""
    cfg = synth.SyncConfig("flat", (4,), (10,), "f32", seed=14)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    got_th, got_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    for e in range(4):
        sl = slice(10 * e, 10 * e + 10)
        delta = th[sl].astype(np.float64) - ps[e].astype(np.float64)
        want = th[sl] - LR * (1 + MU) * delta
        assert np.all(np.abs(got_th[sl] - want) <= one_ulp(want))
        assert np.all(np.abs(got_mo[sl] - delta) <= one_ulp(delta))


def test_modules_are_independent_and_labels_permute():
    cfg = tiny_cfg((1, 3, 2), (5, 8, 6), momentum_std=1e-2, seed=15)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    base_th, base_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    # disturb the level-2 slot of the paths through level-2 module 1: only that module changes
    ps2 = [p.copy() for p in ps]
    touched = [i for i in range(cfg.num_paths) if pr.table[i, 1] == 1]
    for i in touched:
        ps2[i][5:13] += np.float32(0.5)
    th2, mo2, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps2)
    changed = np.nonzero(th2 != base_th)[0]
    assert changed.min() >= 5 + 8 and changed.max() < 5 + 16
    # relabel level-2 modules with a permutation: outputs move with the labels
    perm = np.array([2, 0, 1])
    table_p = pr.table.copy()
    table_p[:, 1] = perm[pr.table[:, 1]]
    th_p = th.copy()
    mo_p = mo.copy()
    for e in range(3):
        th_p[5 + 8 * perm[e]:5 + 8 * perm[e] + 8] = th[5 + 8 * e:5 + 8 * e + 8]
        mo_p[5 + 8 * perm[e]:5 + 8 * perm[e] + 8] = mo[5 + 8 * e:5 + 8 * e + 8]
    th3, mo3, _ = helpers.run_oracle(cfg, table_p, th_p, mo_p, ps)
    for e in range(3):
        np.testing.assert_array_equal(th3[5 + 8 * perm[e]:5 + 8 * perm[e] + 8],
                                      base_th[5 + 8 * e:5 + 8 * e + 8])


# ---------------------------------------------------------------------------- write-back, mask

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_after_sync_every_copy_of_a_module_is_the_new_global_value(dtype):
    cfg = tiny_cfg((1, 2, 2), (7, 9, 4), dtype, seed=16)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    reported = np.array([1, 0, 1, 1], dtype=np.uint8)
    got_th, _, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, None, reported)
    for (l, e, ts, psl) in module_slices(cfg):
        for i in range(cfg.num_paths):
            if pr.table[i, l] != e:
                continue
            if dtype == "bf16":
                want = helpers.float_to_bf16_bits_torch(got_th[ts])
            else:
                want = got_th[ts]
            np.testing.assert_array_equal(got_ps[i][psl], want)


def test_masked_paths_data_is_never_read():
    cfg = tiny_cfg((1, 2, 2), (6, 6, 6), seed=17)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    reported = np.array([1, 0, 1, 1], dtype=np.uint8)
    a = helpers.run_oracle(cfg, pr.table, th, mo, ps, None, reported)
    ps_bad = [p.copy() for p in ps]
    ps_bad[1][:] = np.nan
    b = helpers.run_oracle(cfg, pr.table, th, mo, ps_bad, None, reported)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])
    for x, y in zip(a[2], b[2]):
        np.testing.assert_array_equal(x, y)


def test_bf16_cast_is_round_to_nearest_even_like_the_library_cast():
    vals = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8,
                     -1.0 - 2 ** -8, 3.0e38, 3.4e38, 1e-40, -0.0, np.inf, -np.inf],
                    dtype=np.float32)
    rng = np.random.RandomState(0)
    vals = np.concatenate([vals, rng.normal(0, 0.02, 4096).astype(np.float32),
                           rng.randint(0, 2 ** 31 - 2 ** 24, 4096).astype(np.uint32).view(np.float32)])
    vals = vals[np.isfinite(vals) | np.isinf(vals)]
    n = vals.size
    cfg = synth.SyncConfig("cast", (1,), (n,), "bf16")
    table = np.zeros((1, 1), dtype=np.int32)
    # lr = 1, mu = 0, one path whose copy is exactly representable: theta' = that copy;
    # instead drive theta' directly: no reporter => copies are reset to cast(theta)
    th, mo, ps = helpers.run_oracle(cfg, table, vals, np.zeros(n, np.float32),
                                    [np.zeros(n, np.uint16)], None, np.zeros(1, np.uint8))
    np.testing.assert_array_equal(ps[0], helpers.float_to_bf16_bits_torch(vals))


def test_bf16_cast_of_nan_is_a_nan_whatever_its_payload():
    """A NaN module value reaches the copies as a NaN: never as an infinity (what rounding the
    bit pattern like a number gives when the payload sits in the low 16 bits only) and never as a
    finite value.  Which NaN (sign, payload) is not specified, exactly as for the library cast,
    which returns its canonical quiet NaN."""
    bits = np.array([0x7fc00000, 0xffc00000, 0x7f800001, 0xff800001, 0x7f80ffff, 0x7fffffff,
                     0x7f808000, 0x7fa00000, 0xffffffff, 0x7fc00001], dtype=np.uint32)
    vals = bits.view(np.float32)
    assert np.all(np.isnan(vals))
    n = vals.size
    cfg = synth.SyncConfig("nan", (1,), (n,), "bf16")
    table = np.zeros((1, 1), dtype=np.int32)
    # nobody reports: theta is kept and every copy receives cast(theta)
    th, mo, ps = helpers.run_oracle(cfg, table, vals, np.zeros(n, np.float32),
                                    [np.zeros(n, np.uint16)], None, np.zeros(1, np.uint8))
    np.testing.assert_array_equal(th.view(np.uint32), bits)
    out = ps[0].astype(np.uint32)
    assert np.all((out & 0x7f80) == 0x7f80) and np.all((out & 0x007f) != 0)
    lib = helpers.bf16_bits_to_float(helpers.float_to_bf16_bits_torch(vals))
    assert np.all(np.isnan(lib)) and np.all(np.isnan(helpers.bf16_bits_to_float(ps[0])))


def test_threads_do_not_change_the_result():
    cfg = tiny_cfg((1, 2, 2), (1000, 777, 513), "bf16", momentum_std=1e-3, seed=18)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    a = helpers.run_oracle(cfg, pr.table, th, mo, ps, num_threads=1)
    b = helpers.run_oracle(cfg, pr.table, th, mo, ps, num_threads=4)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])
    for x, y in zip(a[2], b[2]):
        np.testing.assert_array_equal(x, y)


def test_rejects_a_table_entry_out_of_range():
    cfg = tiny_cfg((1, 2), (4, 4))
    table = synth.path_table(cfg.modules_per_level).copy()
    table[1, 1] = 2
    th = np.zeros(cfg.module_params, np.float32)
    with pytest.raises(ValueError):
        oracle.outer_sync(cfg.modules_per_level, cfg.level_numel, table, th, th.copy(),
                          [np.zeros(8, np.float32) for _ in range(2)], oracle.F32, LR, MU)


# ---------------------------------------------------------------------------- Section 2.7 options

def test_module_scale_multiplies_the_outer_gradient():
    """Delta <- s * Delta: with m = 0 the new momentum is s times the unscaled one; with lr = 1,
    mu = 0 theta' = theta - s * (theta - mean); s = 0 leaves theta and only decays momentum."""
    cfg = tiny_cfg((1, 2, 2), (6, 5, 7), seed=21)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    scale = np.array([2.0, 0.5, 4.0, 1.0, 0.0])          # one per module, level-major
    _, base_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    got_th, got_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, module_scale=scale)
    mean_th, _, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, lr=1.0, mu=0.0, module_scale=scale)
    for idx, (l, e, ts, psl) in enumerate(module_slices(cfg)):
        np.testing.assert_allclose(got_mo[ts], scale[idx] * base_mo[ts].astype(np.float64),
                                   rtol=2e-7, atol=0)
        S = [i for i in range(cfg.num_paths) if pr.table[i, l] == e]
        mean = np.mean(np.stack([ps[i][psl].astype(np.float64) for i in S]), axis=0)
        want = th[ts] - scale[idx] * (th[ts].astype(np.float64) - mean)
        assert np.all(np.abs(mean_th[ts] - want) <= one_ulp(want))
    last = module_slices(cfg)[-1][2]
    np.testing.assert_array_equal(got_th[last], th[last])   # s = 0, m = 0: nothing moves
    ones = helpers.run_oracle(cfg, pr.table, th, mo, ps, module_scale=np.ones(5))
    plain = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    np.testing.assert_array_equal(ones[0], plain[0])
    np.testing.assert_array_equal(ones[1], plain[1])


def test_levels_flagged_as_not_communicated_are_left_untouched():
    cfg = tiny_cfg((1, 2, 2), (6, 5, 7), "bf16", momentum_std=1e-2, seed=22)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    flags = np.array([1, 0, 1], dtype=np.uint8)
    got_th, got_mo, got_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps, level_sync=flags)
    full_th, full_mo, full_ps = helpers.run_oracle(cfg, pr.table, th, mo, ps)
    skipped = slice(6, 16)          # the two level-2 modules of 5 parameters each
    np.testing.assert_array_equal(got_th[skipped], th[skipped])
    np.testing.assert_array_equal(got_mo[skipped], mo[skipped])
    for i in range(cfg.num_paths):
        np.testing.assert_array_equal(got_ps[i][6:11], ps[i][6:11])       # copies keep their own values
        np.testing.assert_array_equal(got_ps[i][:6], full_ps[i][:6])
        np.testing.assert_array_equal(got_ps[i][11:], full_ps[i][11:])
    np.testing.assert_array_equal(got_th[:6], full_th[:6])
    np.testing.assert_array_equal(got_th[16:], full_th[16:])
    np.testing.assert_array_equal(got_mo[16:], full_mo[16:])


# ---------------------------------------------------------------------------- other outer optimisers

@pytest.mark.parametrize("kind,nesterov", [(oracle.MOMENTUM, False), (oracle.NESTEROV, True)])
def test_momentum_variants_match_the_library_sgd(kind, nesterov):
    """Three rounds against torch.optim.SGD(momentum, nesterov=...) fed with numpy's mean."""
    cfg = synth.SyncConfig("dense", (1,), (129,), "f32")
    table = np.zeros((4, 1), dtype=np.int32)
    rng = np.random.RandomState(4)
    theta = rng.normal(0, 0.02, 129).astype(np.float32)
    momentum = np.zeros(129, dtype=np.float32)
    param = torch.nn.Parameter(torch.from_numpy(theta.copy()).double())
    opt = torch.optim.SGD([param], lr=LR, momentum=MU, nesterov=nesterov)
    for rnd in range(3):
        paths = [(theta + rng.normal(0, 1e-3, 129)).astype(np.float32) for _ in range(4)]
        delta = np.mean(np.stack([theta.astype(np.float64) - p.astype(np.float64) for p in paths]), axis=0)
        with torch.no_grad():
            param.copy_(torch.from_numpy(theta.astype(np.float64)))
        if rnd > 0:   # the oracle keeps its momentum in fp32: start the library step from the same state
            opt.state[param]["momentum_buffer"] = torch.from_numpy(momentum.astype(np.float64))
        param.grad = torch.from_numpy(delta.copy())
        opt.step()
        theta, momentum, _ = helpers.run_oracle(cfg, table, theta, momentum, paths, optimizer=kind)
        want = param.detach().numpy()
        assert np.all(np.abs(theta - want) <= one_ulp(want))


def test_heavy_ball_constant_gradient_series_and_plain_sgd():
    cfg = tiny_cfg((1,), (2,))
    table = synth.path_table(cfg.modules_per_level)
    theta = np.array([4.0, -1.0], dtype=np.float32)
    momentum = np.zeros(2, dtype=np.float32)
    # heavy ball under g = 1: m_T = (1 - mu^T)/(1 - mu), step_T = lr * m_T  -> 0.7, 1.33, 1.897
    for want_step in (0.7, 1.33, 1.897):
        new_th, momentum, _ = helpers.run_oracle(cfg, table, theta, momentum, [theta - np.float32(1.0)],
                                                 optimizer=oracle.MOMENTUM)
        np.testing.assert_allclose(theta - new_th, want_step, rtol=0, atol=4e-6)
        theta = new_th
    # plain SGD with lr = 1 is the mean of the copies and leaves the momentum buffer alone
    cfg = tiny_cfg((1, 2), (5, 4), momentum_std=1e-2, seed=31)
    pr = synth.make_problem(cfg)
    th, mo, ps = helpers.host_copy(pr)
    got_th, got_mo, _ = helpers.run_oracle(cfg, pr.table, th, mo, ps, lr=1.0, optimizer=oracle.SGD)
    np.testing.assert_array_equal(got_mo, mo)
    want = np.mean(np.stack([p[:5].astype(np.float64) for p in ps]), axis=0)
    assert np.all(np.abs(got_th[:5] - want) <= one_ulp(want))
    with pytest.raises(ValueError):
        helpers.run_oracle(cfg, pr.table, th, mo, ps, optimizer=3)


# ---------------------------------------------------------------------------- Adam family, gradients

def test_adam_family_matches_library_adamw_on_aggregated_gradients():
    """The synchronous variant: path buffers hold gradients, the module-wise weighted mean of them
    drives bias-corrected AdamW.  Three steps against torch.optim.AdamW."""
    cfg = synth.SyncConfig("dense", (1,), (97,), "f32")
    table = np.zeros((3, 1), dtype=np.int32)
    rng = np.random.RandomState(8)
    theta = rng.normal(0, 0.02, 97).astype(np.float32)
    m = np.zeros(97, dtype=np.float32)
    v = np.zeros(97, dtype=np.float32)
    lr, b1, b2, eps, wd = 4e-4, 0.9, 0.999, 1e-8, 0.1
    weights = np.array([3.0, 1.0, 4.0], dtype=np.float32)
    param = torch.nn.Parameter(torch.from_numpy(theta.copy()).double())
    opt = torch.optim.AdamW([param], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    for t in range(1, 4):
        grads = [rng.normal(0, 1e-2, 97).astype(np.float32) for _ in range(3)]
        g = np.average(np.stack(grads).astype(np.float64), axis=0, weights=weights.astype(np.float64))
        with torch.no_grad():
            param.copy_(torch.from_numpy(theta.astype(np.float64)))
        if t > 1:   # the oracle keeps its state in fp32: start the library step from the same state
            opt.state[param]["exp_avg"] = torch.from_numpy(m.astype(np.float64))
            opt.state[param]["exp_avg_sq"] = torch.from_numpy(v.astype(np.float64))
        param.grad = torch.from_numpy(g.copy())
        opt.step()
        adam = (b1, b2, eps, wd, 1 - b1 ** t, 1 - b2 ** t)
        bufs = [x.copy() for x in grads]
        theta, m, bufs = helpers.run_oracle(cfg, table, theta, m, bufs, weights, None, lr=lr,
                                            optimizer=oracle.ADAM, second_moment=v, adam=adam,
                                            input_kind=oracle.GRADIENTS)
        want = param.detach().numpy()
        assert np.all(np.abs(theta - want) <= one_ulp(want))
        np.testing.assert_allclose(m, opt.state[param]["exp_avg"].numpy(), rtol=2e-7, atol=1e-45)
        np.testing.assert_allclose(v, opt.state[param]["exp_avg_sq"].numpy(), rtol=2e-7, atol=1e-45)
        for b in bufs:      # the buffers now hold the new parameters
            np.testing.assert_array_equal(b, theta)


def test_federated_adam_closed_forms_on_outer_gradients():
    """No bias correction, no decay: from m = v = 0 the first step is
    lr*(1-b1)*Delta / (sqrt(1-b2)*|Delta| + tau); with b1 = b2 = 0 it is lr*Delta/(|Delta| + tau);
    a constant outer gradient drives the step towards lr*g/(|g| + tau)."""
    cfg = tiny_cfg((1,), (6,))
    table = synth.path_table(cfg.modules_per_level)
    theta = np.array([1.0, -2.0, 0.5, 3.0, -0.25, 8.0], dtype=np.float32)
    delta = np.array([0.5, -0.25, 0.125, 1.0, -2.0, 0.0], dtype=np.float32)
    zeros = np.zeros(6, dtype=np.float32)
    lr, tau = 0.1, 1e-3
    for b1, b2 in ((0.9, 0.99), (0.0, 0.0)):
        v = zeros.copy()
        th, m, _ = helpers.run_oracle(cfg, table, theta, zeros, [theta - delta], lr=lr,
                                      optimizer=oracle.ADAM, second_moment=v, adam=(b1, b2, tau, 0, 1, 1))
        d = delta.astype(np.float64)
        want = theta - lr * (1 - b1) * d / (np.sqrt(1 - b2) * np.abs(d) + tau)
        assert np.all(np.abs(th - want) <= one_ulp(want))
        np.testing.assert_allclose(m, (1 - b1) * d, rtol=2e-7)
        np.testing.assert_allclose(v, (1 - b2) * d * d, rtol=2e-7)
    th, m, v = theta.copy(), zeros.copy(), zeros.copy()
    for _ in range(400):
        prev = th
        th, m, _ = helpers.run_oracle(cfg, table, th, m, [th - delta], lr=lr, optimizer=oracle.ADAM,
                                      second_moment=v, adam=(0.9, 0.9, tau, 0, 1, 1))
    d = delta.astype(np.float64)
    np.testing.assert_allclose(prev - th, lr * d / (np.abs(d) + tau), rtol=1e-4, atol=1e-6)
    # gradients as inputs with plain SGD: theta' = theta - lr * weighted mean of the gradients
    g = [np.full(6, 2.0, np.float32), np.full(6, 4.0, np.float32)]
    th, _, _ = helpers.run_oracle(cfg, np.zeros((2, 1), np.int32), theta, zeros, g, lr=0.5,
                                  optimizer=oracle.SGD, input_kind=oracle.GRADIENTS)
    np.testing.assert_array_equal(th, theta - np.float32(1.5))
    with pytest.raises(ValueError):
        helpers.run_oracle(cfg, table, theta, zeros, [theta.copy()], optimizer=oracle.ADAM)
