"""Seeded synthetic inputs for the outer synchronisation (no arithmetic of the method here).

The workloads mirror the shapes of the paper's experiments (Section 4: paths of about 150M
parameters; Section 2.6.2: a 16x16 mixture has 256 paths): a first level with one module that
every path shares (Figure "DiPaCo", level 1), followed by levels with K_l modules each.  Path
ids enumerate the product of the levels row-major, last level fastest (Section 2.2 collapses
[j_1..j_L] into one index j).

Values: module parameters theta ~ N(0, 0.02^2); every path's copy of a module is
theta + N(0, 1e-3^2) drawn independently per path (standing in for tau inner steps of
training), stored as fp32 or rounded to bf16; momentum zero or N(0, 1e-4^2).  Weights are
uniform, integer token counts U[1000, 10000], or Zipf(s=1.1) counts; the mask of paths that did
not report is Bernoulli.

This module only produces inputs.  Both the CUDA tests and the CPU oracle tests use it, and it
imports neither of them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class SyncConfig:
    name: str
    modules_per_level: Sequence[int]          # K_l
    level_numel: Sequence[int]                # |B_l|
    path_dtype: str = "f32"                   # "f32" | "bf16"
    weights: str = "uniform"                  # "uniform" | "tokens" | "zipf"
    mask_prob: float = 0.0                    # P(path did not report)
    theta_std: float = 0.02
    delta_std: float = 1e-3
    momentum_std: float = 0.0
    outlier_frac: float = 0.0                 # fraction of delta entries multiplied by outlier_scale
    outlier_scale: float = 100.0
    chunk_paths: int = 0                      # paths per chunk when streamed; 0 = all resident
    outer_lr: float = 0.7
    outer_momentum: float = 0.9
    seed: int = 0

    @property
    def num_levels(self) -> int:
        return len(self.modules_per_level)

    @property
    def num_paths(self) -> int:
        return int(np.prod(self.modules_per_level))

    @property
    def params_per_path(self) -> int:
        return int(sum(self.level_numel))

    @property
    def module_params(self) -> int:
        return int(sum(k * n for k, n in zip(self.modules_per_level, self.level_numel)))

    @property
    def path_params(self) -> int:
        return self.num_paths * self.params_per_path

    def scaled(self, level_numel: Sequence[int], name: Optional[str] = None) -> "SyncConfig":
        """Same grid, weights, mask and value recipe with other module sizes."""
        assert len(level_numel) == self.num_levels
        return dataclasses.replace(self, level_numel=tuple(int(n) for n in level_numel),
                                   name=name or (self.name + "-scaled"))


# The five workloads.  "M" in configs 1-2 is a power of two, in 3-5 a decimal million (150e6
# parameters per path as in the paper's Section 4).
CONFIGS = {
    "grid2x2": SyncConfig("grid2x2", (1, 2, 2), (16384, 65536, 65536), "f32"),
    "grid4x4": SyncConfig("grid4x4", (1, 4, 4), (4194304, 1048576, 1048576), "f32",
                          weights="tokens", momentum_std=1e-4),
    "grid16x16": SyncConfig("grid16x16", (1, 16, 16), (50_000_000,) * 3, "bf16", chunk_paths=32),
    "grid16x16-masked": SyncConfig("grid16x16-masked", (1, 16, 16), (50_000_000,) * 3, "bf16",
                                   weights="zipf", mask_prob=0.2, chunk_paths=32),
    "grid4x4x4x4": SyncConfig("grid4x4x4x4", (1, 4, 4, 4, 4), (20_000_000,) + (10_000_000,) * 4,
                              "bf16", outlier_frac=0.01),
    # the 16x16 grid with an odd level size: every module of theta after the first and every slot
    # of a path copy starts inside a 16-byte unit, and copies that are rows of one block sit at all
    # eight positions within a unit
    "grid16x16-odd-level-size": SyncConfig("grid16x16-odd-level-size", (1, 16, 16), (20_000_003,) * 3,
                                           "bf16", chunk_paths=32),
}


def path_table(modules_per_level: Sequence[int]) -> np.ndarray:
    """[P, L] int32: the module that path j uses at each level (row-major, last level fastest)."""
    K = [int(k) for k in modules_per_level]
    P = int(np.prod(K))
    table = np.zeros((P, len(K)), dtype=np.int32)
    for j in range(P):
        rem = j
        for l in range(len(K) - 1, -1, -1):
            table[j, l] = rem % K[l]
            rem //= K[l]
    return table


def path_weights(cfg: SyncConfig) -> Optional[np.ndarray]:
    """Raw per-path weights (token counts) as float32, or None for uniform."""
    P = cfg.num_paths
    rng = np.random.RandomState(cfg.seed + 101)
    if cfg.weights == "uniform":
        return None
    if cfg.weights == "tokens":
        return rng.randint(1000, 10001, size=P).astype(np.float32)
    if cfg.weights == "zipf":
        rank = rng.permutation(P) + 1
        return np.ceil(1e7 / rank.astype(np.float64) ** 1.1).astype(np.float32)
    raise ValueError(cfg.weights)


def reported_mask(cfg: SyncConfig) -> Optional[np.ndarray]:
    """uint8 [P], 1 = the path reported; None when every path reports."""
    if cfg.mask_prob <= 0.0:
        return None
    rng = np.random.RandomState(cfg.seed + 202)
    return (rng.random_sample(cfg.num_paths) >= cfg.mask_prob).astype(np.uint8)


@dataclasses.dataclass
class SyncProblem:
    cfg: SyncConfig
    table: np.ndarray                     # [P, L] int32
    weights: Optional[np.ndarray]         # [P] float32 or None
    reported: Optional[np.ndarray]        # [P] uint8 or None
    theta: torch.Tensor                   # fp32 [module_params]
    momentum: torch.Tensor                # fp32 [module_params]
    paths: List[torch.Tensor]             # P tensors [params_per_path], fp32 or bf16
    storage: Optional[torch.Tensor] = None  # the [P, params_per_path] block behind `paths`, if any

    def module_offsets(self) -> np.ndarray:
        """[L+1] offsets of each level's first module inside theta / momentum."""
        sizes = [k * n for k, n in zip(self.cfg.modules_per_level, self.cfg.level_numel)]
        return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)

    def level_offsets(self) -> np.ndarray:
        """[L+1] offsets of each level inside one path copy."""
        return np.concatenate([[0], np.cumsum(self.cfg.level_numel)]).astype(np.int64)


def torch_path_dtype(cfg: SyncConfig) -> torch.dtype:
    return torch.bfloat16 if cfg.path_dtype == "bf16" else torch.float32


def make_problem(cfg: SyncConfig, device="cpu", separate_buffers: bool = False,
                 pin_paths: bool = False) -> SyncProblem:
    """Draw theta, momentum and the P path copies on `device` from cfg.seed."""
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed)
    table = path_table(cfg.modules_per_level)
    P, L = table.shape
    total = cfg.module_params
    theta = torch.empty(total, dtype=torch.float32, device=device)
    theta.normal_(0.0, cfg.theta_std, generator=gen)
    momentum = torch.zeros(total, dtype=torch.float32, device=device)
    if cfg.momentum_std > 0.0:
        momentum.normal_(0.0, cfg.momentum_std, generator=gen)

    dt = torch_path_dtype(cfg)
    per_path = cfg.params_per_path
    storage = None
    if separate_buffers:
        paths = [torch.empty(per_path, dtype=dt, device=device) for _ in range(P)]
    else:
        storage = torch.empty((P, per_path), dtype=dt, device=device,
                              pin_memory=(pin_paths and device.type == "cpu"))
        paths = [storage[i] for i in range(P)]

    mod_off = np.concatenate(
        [[0], np.cumsum([k * n for k, n in zip(cfg.modules_per_level, cfg.level_numel)])])
    lvl_off = np.concatenate([[0], np.cumsum(cfg.level_numel)])
    for i in range(P):
        for l in range(L):
            n = int(cfg.level_numel[l])
            if n == 0:
                continue
            src = int(mod_off[l]) + int(table[i, l]) * n
            delta = torch.empty(n, dtype=torch.float32, device=device)
            delta.normal_(0.0, cfg.delta_std, generator=gen)
            if cfg.outlier_frac > 0.0:
                pick = torch.empty(n, dtype=torch.float32, device=device)
                pick.uniform_(0.0, 1.0, generator=gen)
                delta = torch.where(pick < cfg.outlier_frac, delta * cfg.outlier_scale, delta)
            delta.add_(theta[src:src + n])
            paths[i][int(lvl_off[l]):int(lvl_off[l]) + n].copy_(delta)
    return SyncProblem(cfg, table, path_weights(cfg), reported_mask(cfg), theta, momentum, paths,
                       storage)


def algorithmic_bytes(cfg: SyncConfig, reported: Optional[np.ndarray] = None) -> int:
    """Bytes one synchronisation has to move: each reporting copy read once, every copy written
    once, theta and momentum (fp32) read and written once."""
    s = 2 if cfg.path_dtype == "bf16" else 4
    n_rep = cfg.num_paths if reported is None else int(np.asarray(reported).sum())
    return (n_rep + cfg.num_paths) * cfg.params_per_path * s + 16 * cfg.module_params
