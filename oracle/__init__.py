"""Loader for the CPU oracle of DiPaCo's outer synchronisation (Algorithm 1, outer loop).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the CPU-baseline
leg of the benchmark.  Nothing in the CUDA library or its Python binding imports this package,
and this package imports nothing from them.

The arithmetic lives in ``outer_sync_oracle.c`` (plain C, double precision); this file only
compiles it with gcc and marshals numpy arrays into its one entry point.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "outer_sync_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32 = 0
BF16 = 1

NESTEROV = 0
MOMENTUM = 1
SGD = 2
ADAM = 3

COPIES = 0
GRADIENTS = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``); returns the path of the shared object."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_outer_sync.restype = ctypes.c_int
        lib.oracle_outer_sync.argtypes = [
            ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_double, ctypes.c_double, ctypes.c_int32,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
        ]
        lib.oracle_outer_sync_ex.restype = ctypes.c_int
        lib.oracle_outer_sync_ex.argtypes = lib.oracle_outer_sync.argtypes + [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32]
        lib.oracle_max_threads.restype = ctypes.c_int32
        lib.oracle_max_threads.argtypes = []
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def outer_sync(modules_per_level, level_numel, path_to_module, theta, momentum, paths,
               path_dtype, outer_lr, outer_momentum, path_weights=None, reported=None,
               num_threads=1, module_scale=None, level_sync=None, optimizer=NESTEROV,
               second_moment=None, adam=None, input_kind=COPIES):
    """Run one outer synchronisation in place on host arrays.

    theta, momentum: contiguous float32 numpy arrays of sum_l K_l*N_l elements (level, module,
    element order).  paths: list of P contiguous numpy arrays, float32 for ``F32`` or uint16
    (raw bf16 bits) for ``BF16``, each of sum_l N_l elements.  path_to_module: int array [P, L].
    path_weights: None (uniform) or [P] float32.  reported: None (all) or [P] of 0/1.
    module_scale: None or [sum_l K_l] factors on the modules' outer gradients (level-major).
    level_sync: None or [L] of 0/1, 0 = the level is left untouched.
    optimizer: NESTEROV (the paper's), MOMENTUM (heavy ball), SGD or ADAM.
    second_moment: float32 array like theta (ADAM only).  adam: (b1, b2, eps, weight_decay, c1, c2).
    input_kind: COPIES, or GRADIENTS when the path buffers hold gradients instead of copies.
    """
    lib = _load()
    K = np.ascontiguousarray(modules_per_level, dtype=np.int32)
    N = np.ascontiguousarray(level_numel, dtype=np.int64)
    table = np.ascontiguousarray(path_to_module, dtype=np.int32)
    L = int(K.shape[0])
    P = int(table.shape[0])
    assert table.shape == (P, L) and N.shape == (L,)
    total = int((K.astype(np.int64) * N).sum())
    per_path = int(N.sum())
    want = np.float32 if path_dtype == F32 else np.uint16
    for a in (theta, momentum):
        assert a.dtype == np.float32 and a.flags.c_contiguous and a.size == total
    assert len(paths) == P
    for p in paths:
        assert p.dtype == want and p.flags.c_contiguous and p.size == per_path
    ptrs = (ctypes.c_void_p * P)(*[p.ctypes.data for p in paths])
    w = None
    if path_weights is not None:
        w = np.ascontiguousarray(path_weights, dtype=np.float32)
        assert w.shape == (P,)
    r = None
    if reported is not None:
        r = np.ascontiguousarray(reported, dtype=np.uint8)
        assert r.shape == (P,)
    sc = None
    if module_scale is not None:
        sc = np.ascontiguousarray(module_scale, dtype=np.float64)
        assert sc.shape == (int(K.sum()),)
    ls = None
    if level_sync is not None:
        ls = np.ascontiguousarray(level_sync, dtype=np.uint8)
        assert ls.shape == (L,)
    ad = None
    if adam is not None:
        ad = np.ascontiguousarray(adam, dtype=np.float64)
        assert ad.shape == (6,)
    if second_moment is not None:
        assert second_moment.dtype == np.float32 and second_moment.flags.c_contiguous
        assert second_moment.size == total
    rc = lib.oracle_outer_sync_ex(
        L, K.ctypes.data, N.ctypes.data, P, table.ctypes.data,
        w.ctypes.data if w is not None else None,
        r.ctypes.data if r is not None else None,
        float(outer_lr), float(outer_momentum), int(path_dtype),
        theta.ctypes.data, momentum.ctypes.data, ctypes.cast(ptrs, ctypes.c_void_p),
        int(num_threads),
        sc.ctypes.data if sc is not None else None,
        ls.ctypes.data if ls is not None else None,
        int(optimizer),
        second_moment.ctypes.data if second_moment is not None else None,
        ad.ctypes.data if ad is not None else None,
        int(input_kind),
    )
    if rc != 0:
        raise ValueError("oracle_outer_sync rejected its arguments")
