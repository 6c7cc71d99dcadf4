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
