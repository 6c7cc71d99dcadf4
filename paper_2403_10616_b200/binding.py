"""ctypes binding of ``libdipaco.so`` (declared in ``include/dipaco.h``).

Argument marshalling only: every step of the synchronisation runs in the CUDA library.  The
functions carry the names of the C entry points; ``OuterSync`` is a thin owner of one context.
Tensors are torch tensors used as device (or pinned host) memory; streams are torch streams.
There is no fallback: a missing library raises at load time.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdipaco.so")

DIPACO_F32 = 0
DIPACO_BF16 = 1

DIPACO_OK = 0
DIPACO_EINVAL = -1
DIPACO_ECUDA = -2
DIPACO_ENOMEM = -3
DIPACO_ESTATE = -4
DIPACO_ETIMEOUT = -5
DIPACO_ENODEV = -6
DIPACO_ELIMIT = -7
DIPACO_STATIC_MAX_NUMEL = 4 * 1024 * 1024

DIPACO_OPT_NESTEROV = 0
DIPACO_OPT_MOMENTUM = 1
DIPACO_OPT_SGD = 2
DIPACO_OPT_ADAM = 3

DIPACO_INPUT_COPIES = 0
DIPACO_INPUT_GRADIENTS = 1

DIPACO_KERNEL_AUTO = 0
DIPACO_KERNEL_VECTOR = 1
DIPACO_KERNEL_SCALAR = 2

EXPORTS = [
    "dipaco_create", "dipaco_outer_sync", "dipaco_destroy", "dipaco_strerror",
    "dipaco_sync_begin", "dipaco_sync_accumulate", "dipaco_sync_writeback", "dipaco_sync_end",
    "dipaco_outer_sync_host", "dipaco_set_weights", "dipaco_set_kernel", "dipaco_set_tuning",
    "dipaco_device_status", "dipaco_launch_count", "dipaco_plan_module", "dipaco_plan_offsets",
    "dipaco_plan_chunks", "dipaco_plan_split", "dipaco_module_sync_static",
    "dipaco_set_host_unit_bytes", "dipaco_plan_traffic", "dipaco_set_module_scale",
    "dipaco_set_level_sync", "dipaco_set_shard", "dipaco_set_optimizer", "dipaco_set_adam",
    "dipaco_set_input_kind", "dipaco_plan_shard", "dipaco_create_shard",
    "dipaco_selftest_wait_expiry", "dipaco_set_work_items", "dipaco_set_host_threads",
]

_lib = None


class DipacoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, strerror(status), status))


def load() -> ctypes.CDLL:
    """Load libdipaco.so; raises if it has not been built (``python -m paper_2403_10616_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "CUDA library %s is missing: build it with `python -m paper_2403_10616_b200.build`; "
            "there is no CPU fallback" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.dipaco_create.argtypes = [ctypes.POINTER(vp), i32, vp, vp, i32, vp, vp, f32, f32, i32, i32, i32]
    lib.dipaco_outer_sync.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dipaco_destroy.argtypes = [vp]
    lib.dipaco_strerror.argtypes = [ctypes.c_int]
    lib.dipaco_strerror.restype = ctypes.c_char_p
    lib.dipaco_sync_begin.argtypes = [vp, vp, vp, vp, vp]
    lib.dipaco_sync_accumulate.argtypes = [vp, i32, vp]
    lib.dipaco_sync_writeback.argtypes = [vp, i32, vp]
    lib.dipaco_sync_end.argtypes = [vp]
    lib.dipaco_outer_sync_host.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dipaco_set_weights.argtypes = [vp, vp]
    lib.dipaco_set_module_scale.argtypes = [vp, vp]
    lib.dipaco_set_level_sync.argtypes = [vp, vp]
    lib.dipaco_set_shard.argtypes = [vp, i32, i32]
    lib.dipaco_plan_shard.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.dipaco_create_shard.argtypes = [ctypes.POINTER(vp), vp, i32, i32, i32]
    lib.dipaco_selftest_wait_expiry.argtypes = [vp, i64, vp]
    lib.dipaco_set_optimizer.argtypes = [vp, i32]
    lib.dipaco_set_adam.argtypes = [vp, vp, f32, f32, f32, f32, i32]
    lib.dipaco_set_input_kind.argtypes = [vp, i32]
    lib.dipaco_set_kernel.argtypes = [vp, i32]
    lib.dipaco_set_tuning.argtypes = [vp, i32, i32, i32, i32]
    lib.dipaco_set_work_items.argtypes = [vp, i64, i32]
    lib.dipaco_set_host_threads.argtypes = [vp, i32]
    lib.dipaco_device_status.argtypes = [vp]
    lib.dipaco_set_host_unit_bytes.argtypes = [vp, i64]
    lib.dipaco_launch_count.argtypes = [vp]
    lib.dipaco_launch_count.restype = i64
    lib.dipaco_plan_module.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.dipaco_plan_offsets.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.dipaco_plan_chunks.argtypes = [vp, vp, vp]
    lib.dipaco_plan_traffic.argtypes = [vp, vp, vp, vp]
    lib.dipaco_plan_split.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp, vp]
    lib.dipaco_module_sync_static.argtypes = [vp, vp, i64, i32, vp, vp, vp, f32, f32, i32, i32, i32, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("dipaco_strerror", "dipaco_launch_count"):
            fn.restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().dipaco_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != DIPACO_OK:
        raise DipacoError(status, where)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _ptr_array(ptrs):
    """A C array of pointers; one that ptr_array() already built is passed through."""
    if isinstance(ptrs, ctypes.Array):
        return ptrs
    return (ctypes.c_void_p * len(ptrs))(*[int(p) for p in ptrs])


def ptr_array(ptrs: Sequence[int]):
    """Build the C pointer array once, for callers that synchronise the same buffers repeatedly."""
    return _ptr_array(ptrs)


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


# ------------------------------------------------------------------ C entry points, same names

def dipaco_create(modules_per_level, level_numel, path_to_module, path_weights=None,
                  outer_lr=0.7, outer_momentum=0.9, path_dtype=DIPACO_F32, chunk_paths=0,
                  device=0) -> int:
    """Returns the context handle (an integer address)."""
    lib = load()
    K = np.ascontiguousarray(modules_per_level, dtype=np.int32)
    N = np.ascontiguousarray(level_numel, dtype=np.int64)
    table = np.ascontiguousarray(path_to_module, dtype=np.int32)
    if table.ndim != 2 or table.shape[1] != K.shape[0] or N.shape != K.shape:
        raise ValueError("path_to_module must be [P, L] with L = len(modules_per_level)")
    w = None if path_weights is None else np.ascontiguousarray(path_weights, dtype=np.float32)
    if w is not None and w.shape != (table.shape[0],):
        raise ValueError("path_weights must have one entry per path")
    handle = ctypes.c_void_p()
    _check(lib.dipaco_create(ctypes.byref(handle), int(K.shape[0]), _np_ptr(K), _np_ptr(N),
                             int(table.shape[0]), _np_ptr(table), _np_ptr(w), float(outer_lr),
                             float(outer_momentum), int(path_dtype), int(chunk_paths), int(device)),
           "dipaco_create")
    return handle.value


def dipaco_destroy(ctx: int) -> None:
    _check(load().dipaco_destroy(ctx), "dipaco_destroy")


def dipaco_outer_sync(ctx: int, theta_ptr: int, momentum_ptr: int, path_ptrs: Sequence[int],
                      reported: Optional[np.ndarray] = None, stream=None) -> None:
    arr = _ptr_array(path_ptrs)
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    _check(load().dipaco_outer_sync(ctx, theta_ptr, momentum_ptr, ctypes.cast(arr, ctypes.c_void_p),
                                    _np_ptr(r), _stream_handle(stream)), "dipaco_outer_sync")


def dipaco_sync_begin(ctx, theta_ptr, momentum_ptr, reported=None, stream=None) -> None:
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    _check(load().dipaco_sync_begin(ctx, theta_ptr, momentum_ptr, _np_ptr(r), _stream_handle(stream)),
           "dipaco_sync_begin")


def dipaco_sync_accumulate(ctx, chunk_index, chunk_ptrs) -> None:
    arr = _ptr_array(chunk_ptrs)
    _check(load().dipaco_sync_accumulate(ctx, int(chunk_index), ctypes.cast(arr, ctypes.c_void_p)),
           "dipaco_sync_accumulate")


def dipaco_sync_writeback(ctx, chunk_index, chunk_ptrs) -> None:
    arr = _ptr_array(chunk_ptrs)
    _check(load().dipaco_sync_writeback(ctx, int(chunk_index), ctypes.cast(arr, ctypes.c_void_p)),
           "dipaco_sync_writeback")


def dipaco_sync_end(ctx) -> None:
    _check(load().dipaco_sync_end(ctx), "dipaco_sync_end")


def dipaco_outer_sync_host(ctx, theta_host_ptr, momentum_host_ptr, path_host_ptrs, reported=None,
                           stream=None) -> None:
    arr = _ptr_array(path_host_ptrs)
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    _check(load().dipaco_outer_sync_host(ctx, theta_host_ptr, momentum_host_ptr,
                                         ctypes.cast(arr, ctypes.c_void_p), _np_ptr(r),
                                         _stream_handle(stream)), "dipaco_outer_sync_host")


def dipaco_set_weights(ctx, path_weights) -> None:
    w = None if path_weights is None else np.ascontiguousarray(path_weights, dtype=np.float32)
    _check(load().dipaco_set_weights(ctx, _np_ptr(w)), "dipaco_set_weights")


def dipaco_set_module_scale(ctx, module_scale) -> None:
    sc = None if module_scale is None else np.ascontiguousarray(module_scale, dtype=np.float32)
    _check(load().dipaco_set_module_scale(ctx, _np_ptr(sc)), "dipaco_set_module_scale")


def dipaco_set_level_sync(ctx, level_sync) -> None:
    ls = None if level_sync is None else np.ascontiguousarray(level_sync, dtype=np.uint8)
    _check(load().dipaco_set_level_sync(ctx, _np_ptr(ls)), "dipaco_set_level_sync")


def dipaco_set_optimizer(ctx, optimizer: int) -> None:
    _check(load().dipaco_set_optimizer(ctx, int(optimizer)), "dipaco_set_optimizer")


def dipaco_set_adam(ctx, second_moment_ptr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0,
                    step=0) -> None:
    _check(load().dipaco_set_adam(ctx, second_moment_ptr, float(beta1), float(beta2), float(eps),
                                  float(weight_decay), int(step)), "dipaco_set_adam")


def dipaco_set_input_kind(ctx, input_kind: int) -> None:
    _check(load().dipaco_set_input_kind(ctx, int(input_kind)), "dipaco_set_input_kind")


def dipaco_set_shard(ctx, shard_index: int, shard_count: int) -> None:
    _check(load().dipaco_set_shard(ctx, int(shard_index), int(shard_count)), "dipaco_set_shard")


def dipaco_plan_shard(ctx, shard_index: int, shard_count: int, level: int):
    """(begin, end): the element range of every module of `level` that the shard owns."""
    a, b = ctypes.c_int64(), ctypes.c_int64()
    _check(load().dipaco_plan_shard(ctx, int(shard_index), int(shard_count), int(level),
                                    ctypes.addressof(a), ctypes.addressof(b)), "dipaco_plan_shard")
    return a.value, b.value


def dipaco_create_shard(whole: int, shard_index: int, shard_count: int, device=0) -> int:
    """Context of one shard in the compact layout; returns its handle."""
    handle = ctypes.c_void_p()
    _check(load().dipaco_create_shard(ctypes.byref(handle), whole, int(shard_index), int(shard_count),
                                      int(device)), "dipaco_create_shard")
    return handle.value


def dipaco_selftest_wait_expiry(ctx, limit_ns: int, stream=None) -> None:
    _check(load().dipaco_selftest_wait_expiry(ctx, int(limit_ns), _stream_handle(stream)),
           "dipaco_selftest_wait_expiry")


def dipaco_set_kernel(ctx, kernel: int) -> None:
    _check(load().dipaco_set_kernel(ctx, int(kernel)), "dipaco_set_kernel")


def dipaco_set_tuning(ctx, ctas_per_sm=0, stages=0, units_per_thread=0, io_slots=0) -> None:
    _check(load().dipaco_set_tuning(ctx, int(ctas_per_sm), int(stages), int(units_per_thread),
                                    int(io_slots)), "dipaco_set_tuning")


def dipaco_set_work_items(ctx, max_item_bytes=0, items_per_cta=0) -> None:
    _check(load().dipaco_set_work_items(ctx, int(max_item_bytes), int(items_per_cta)),
           "dipaco_set_work_items")


def dipaco_set_host_threads(ctx, threads: int) -> None:
    _check(load().dipaco_set_host_threads(ctx, int(threads)), "dipaco_set_host_threads")


def dipaco_set_host_unit_bytes(ctx, nbytes: int) -> None:
    _check(load().dipaco_set_host_unit_bytes(ctx, int(nbytes)), "dipaco_set_host_unit_bytes")


def dipaco_device_status(ctx) -> int:
    return int(load().dipaco_device_status(ctx))


def dipaco_launch_count(ctx) -> int:
    return int(load().dipaco_launch_count(ctx))


def dipaco_plan_module(ctx, level, module, num_paths, reported=None):
    """(members, contributors, coeff, will_update) of one module under a mask."""
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    members = np.zeros(num_paths, dtype=np.int32)
    contributors = np.zeros(num_paths, dtype=np.int32)
    coeff = np.zeros(num_paths, dtype=np.float32)
    nm, nc, upd = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load().dipaco_plan_module(ctx, int(level), int(module), _np_ptr(r),
                                     ctypes.addressof(nm), _np_ptr(members), ctypes.addressof(nc),
                                     _np_ptr(contributors), _np_ptr(coeff), ctypes.addressof(upd)),
           "dipaco_plan_module")
    return members[:nm.value].copy(), contributors[:nc.value].copy(), coeff[:nc.value].copy(), bool(upd.value)


def dipaco_plan_offsets(ctx, level, module):
    a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(load().dipaco_plan_offsets(ctx, int(level), int(module), ctypes.addressof(a),
                                      ctypes.addressof(b), ctypes.addressof(c)), "dipaco_plan_offsets")
    return a.value, b.value, c.value


def dipaco_plan_chunks(ctx):
    n, s = ctypes.c_int32(), ctypes.c_int64()
    _check(load().dipaco_plan_chunks(ctx, ctypes.addressof(n), ctypes.addressof(s)), "dipaco_plan_chunks")
    return n.value, s.value


def dipaco_plan_traffic(ctx, reported=None):
    """(bytes moved by one dipaco_outer_sync by construction, number of launches)."""
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    nbytes, launches = ctypes.c_int64(), ctypes.c_int32()
    _check(load().dipaco_plan_traffic(ctx, _np_ptr(r), ctypes.addressof(nbytes),
                                      ctypes.addressof(launches)), "dipaco_plan_traffic")
    return nbytes.value, launches.value


def dipaco_plan_split(ctx, num_ctas, tile, reported=None, capacity=1 << 16):
    """(seg_level, seg_module, seg_begin, seg_end, cta_first) of the resident-mode launch."""
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    lvl = np.zeros(capacity, dtype=np.int32)
    mod = np.zeros(capacity, dtype=np.int32)
    beg = np.zeros(capacity, dtype=np.int64)
    end = np.zeros(capacity, dtype=np.int64)
    first = np.zeros(num_ctas + 1, dtype=np.int32)
    n = load().dipaco_plan_split(ctx, _np_ptr(r), int(num_ctas), int(tile), int(capacity),
                                 _np_ptr(lvl), _np_ptr(mod), _np_ptr(beg), _np_ptr(end),
                                 _np_ptr(first))
    if n < 0:
        raise DipacoError(n, "dipaco_plan_split")
    return lvl[:n].copy(), mod[:n].copy(), beg[:n].copy(), end[:n].copy(), first


def dipaco_module_sync_static(theta_ptr, momentum_ptr, numel, copy_ptrs, path_weights=None,
                              reported=None, outer_lr=0.7, outer_momentum=0.9,
                              path_dtype=DIPACO_F32, chunk_paths=8, device=0, stream=None) -> None:
    """One module, no allocation: partial sums live in the library's static device array.

    For callers that may not use the device allocator; see the declaration in dipaco.h for the
    size limit, the shared array and the rule about the first call on a device."""
    arr = _ptr_array(copy_ptrs)
    w = None if path_weights is None else np.ascontiguousarray(path_weights, dtype=np.float32)
    r = None if reported is None else np.ascontiguousarray(reported, dtype=np.uint8)
    _check(load().dipaco_module_sync_static(theta_ptr, momentum_ptr, int(numel), len(copy_ptrs),
                                            ctypes.cast(arr, ctypes.c_void_p), _np_ptr(w), _np_ptr(r),
                                            float(outer_lr), float(outer_momentum), int(path_dtype),
                                            int(chunk_paths), int(device), _stream_handle(stream)),
           "dipaco_module_sync_static")


# ------------------------------------------------------------------ convenience owner

class OuterSync:
    """Owns one context.  ``sync(theta, momentum, paths)`` takes torch CUDA tensors."""

    def __init__(self, modules_per_level, level_numel, path_to_module, path_weights=None,
                 outer_lr=0.7, outer_momentum=0.9, path_dtype="f32", chunk_paths=0, device=0):
        self.num_paths = int(np.asarray(path_to_module).shape[0])
        self.path_dtype = path_dtype
        code = DIPACO_BF16 if path_dtype == "bf16" else DIPACO_F32
        self.ctx = dipaco_create(modules_per_level, level_numel, path_to_module, path_weights,
                                 outer_lr, outer_momentum, code, chunk_paths, device)

    @classmethod
    def for_problem(cls, problem, chunk_paths=None, device=0):
        cfg = problem.cfg
        cp = cfg.chunk_paths if chunk_paths is None else chunk_paths
        return cls(cfg.modules_per_level, cfg.level_numel, problem.table, problem.weights,
                   np.float32(cfg.outer_lr), np.float32(cfg.outer_momentum), cfg.path_dtype, cp,
                   device)

    def sync(self, theta, momentum, paths, reported=None, stream=None) -> None:
        dipaco_outer_sync(self.ctx, theta.data_ptr(), momentum.data_ptr(),
                          [p.data_ptr() for p in paths], reported, stream)

    def sync_host(self, theta, momentum, paths, reported=None, stream=None) -> None:
        dipaco_outer_sync_host(self.ctx, theta.data_ptr(), momentum.data_ptr(),
                               [p.data_ptr() for p in paths], reported, stream)

    def status(self) -> int:
        return dipaco_device_status(self.ctx)

    def close(self) -> None:
        if self.ctx is not None:
            ctx, self.ctx = self.ctx, None
            dipaco_destroy(ctx)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
