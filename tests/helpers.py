"""Shared test plumbing: moving a synthetic problem to host arrays and calling the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle


def tensor_to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host copy; bf16 becomes its raw uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def float_to_bf16_bits_torch(x: np.ndarray) -> np.ndarray:
    """bf16 rounding through torch's own cast (a library routine, used to pin the oracle's)."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_step(values: np.ndarray) -> np.ndarray:
    """Spacing of bf16 at each value: 2^(e-7) for a normal value with exponent e, 2^-133 for
    subnormals (bf16 keeps 7 stored significand bits and has fp32's exponent range)."""
    a = np.abs(np.asarray(values, dtype=np.float64))
    _, e = np.frexp(a)                      # a = f * 2^e with f in [0.5, 1)
    e = np.where(a == 0.0, -126, e - 1)
    return np.ldexp(1.0, np.maximum(e, -126) - 7)


def assert_bf16_copies_close(got_bits: np.ndarray, want_bits: np.ndarray, what="a path copy") -> None:
    """Two bf16 roundings of two fp32 values that agree to the fp32 tolerance.

    The fp32 results may differ by 1e-6 * (1 + |x|); rounding each to bf16 can then land on
    neighbouring bf16 values, never further: the allowed distance is the fp32 tolerance plus ONE
    bf16 step at the expected value (the exact spacing there, not a relative bound).  Counting
    differing bit patterns does not work near zero, where the absolute part of the fp32
    tolerance spans many bf16 steps.  NaN must be NaN on both sides (payloads are not compared)."""
    got = bf16_bits_to_float(np.asarray(got_bits)).astype(np.float64)
    want = bf16_bits_to_float(np.asarray(want_bits)).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(nan, np.isnan(got)), what + ": NaN on one side only"
    g, w = got[~nan], want[~nan]
    inf = np.isinf(w)
    assert np.array_equal(g[inf], w[inf]), what + ": infinities differ"
    g, w = g[~inf], w[~inf]
    bound = 1e-6 * (1.0 + np.abs(w)) + bf16_step(w)
    bad = np.abs(g - w) > bound
    assert not bad.any(), "%s is more than one bf16 step (plus the fp32 tolerance) from the oracle's" % what


def host_copy(problem):
    """(theta, momentum, [paths]) as fresh numpy arrays."""
    return (tensor_to_numpy(problem.theta), tensor_to_numpy(problem.momentum),
            [tensor_to_numpy(p) for p in problem.paths])


def run_oracle(cfg, table, theta, momentum, paths, weights=None, reported=None,
               lr=None, mu=None, num_threads=1, module_scale=None, level_sync=None,
               optimizer=0, second_moment=None, adam=None, input_kind=0):
    """Oracle on copies of the given host arrays; returns (theta', m', [copies'])."""
    th = theta.copy()
    mo = momentum.copy()
    ps = [p.copy() for p in paths]
    dtype = oracle.BF16 if cfg.path_dtype == "bf16" else oracle.F32
    lr = np.float32(cfg.outer_lr if lr is None else lr)
    mu = np.float32(cfg.outer_momentum if mu is None else mu)
    oracle.outer_sync(cfg.modules_per_level, cfg.level_numel, table, th, mo, ps, dtype,
                      float(lr), float(mu), weights, reported, num_threads, module_scale, level_sync,
                      optimizer, second_moment, adam, input_kind)
    return th, mo, ps


def path_values(cfg, arr):
    """A path copy as float32 values whatever its storage type."""
    return bf16_bits_to_float(arr) if cfg.path_dtype == "bf16" else arr
