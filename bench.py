#!/usr/bin/env python
"""Benchmark of the module-wise outer synchronisation (DiPaCo, Algorithm 1, outer loop).

One step = one full synchronisation of the 16x16-module, 256-path, 150M-parameters-per-path
workload (bf16 path copies, fp32 module state): outer gradients, segmented reduction over the
paths sharing each module, Nesterov update, write-back into every path.  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "outer_sync_path_params_per_s"
UNIT = "path-params/s"
CPU_SAMPLE_NUMEL = 10_000_000     # parameters per level in the CPU-baseline sample
REF_SAMPLE_NUMEL = 1_000_000      # parameters per level per step in the reference arm


# DRAM traffic of the bulk-copy kernel from the ncu capture summarised under profiles/ (small case of
# the same workload, 2e6 parameters per level): dram__bytes_read.sum + dram__bytes_write.sum divided
# by the algorithmic bytes of that launch.  Traffic grows with the number of tiles, so the full-size
# figure is this ratio times the algorithmic bytes.  Only valid for the sources it was taken from
# (the kernels, the launch code that picks tiles, stages and work items, and the planner): their
# digest is checked and "traffic" is null after any change to them.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 0.9919
NCU_CAPTURE_SOURCES = ("kernels.cuh", "dipaco.cu", "plan.hpp")
NCU_CAPTURE_SOURCES_SHA256 = "63fd72cb32bba49c5bfc6f80f7e446524e0064dc8ead76279df492ad99f8e61d"
NCU_CAPTURE_COMMAND = ("ncu --set full --clock-control none -k regex:sync_bulk_kernel -s 3 -c 3 "
                       "python bench.py --level-numel 2000000 --steps 3 --warmup 3 --no-e2e "
                       "--no-chunked --no-cpu-baseline --no-variants --no-other-workloads")


def sources_digest():
    import hashlib
    h = hashlib.sha256()
    for name in NCU_CAPTURE_SOURCES:
        with open(os.path.join(ROOT, "paper_2403_10616_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="grid16x16")
    ap.add_argument("--level-numel", type=int, default=0,
                    help="override the parameters per level (smaller runs for profiling)")
    ap.add_argument("--mode", default="resident", choices=["resident", "chunked", "adam", "sharded"],
                    help="what the main timed leg runs (the metric is quoted on 'resident'; 'chunked' "
                         "and 'adam' exist to profile the chunk walk and the Adam-family step; "
                         "'sharded' splits the ONE workload over the ranks, rank r updating slab r "
                         "of every module with no exchange: strong scaling)")
    ap.add_argument("--kernel", default="auto", choices=["auto", "vector", "scalar"])
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--units", type=int, default=0)
    ap.add_argument("--io-slots", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--host-unit-mb", type=int, default=0,
                    help="cap on the upload of one streamed unit of the host-buffer leg (0 = default)")
    ap.add_argument("--host-threads", type=int, default=-1,
                    help="host threads that fan each module's result out to its paths in the "
                         "host-buffer leg (-1 = library default, 0 = none: one download per path)")
    ap.add_argument("--items-per-cta", type=int, default=0)
    ap.add_argument("--item-kb", type=int, default=0)
    ap.add_argument("--separate-buffers", action="store_true",
                    help="one allocation per path copy instead of rows of one block (with an odd "
                         "level size the copies then all sit at the same place within a 16-byte unit)")
    ap.add_argument("--no-other-workloads", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-chunked", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true")
    return ap.parse_args()


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU; only the samples that arrive between
    mark_start() and mark_end() (the timed region) are summarised."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        import threading
        self.lines = []
        self.t_start = self.t_end = None
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line))

    def wait_first_sample(self, timeout=10.0):
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < timeout:
            time.sleep(0.02)

    def mark_start(self):
        self.t_start = time.perf_counter()

    def mark_end(self):
        self.t_end = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, power, reasons = [], [], [], set()
        for (t, line) in list(self.lines):
            if self.t_start is not None and not (self.t_start <= t <= (self.t_end or t) + 0.06):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(args):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def aggregate(ms_local, units_local, world, backend_device):
    """(max ms over ranks, total units over ranks); a no-op without torch.distributed."""
    import torch
    import torch.distributed as dist
    if world <= 1 or not dist.is_initialized():
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=backend_device)
    u = torch.tensor([units_local], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier(world):
    import torch.distributed as dist
    if world > 1 and dist.is_initialized():
        dist.barrier()


def workload_config(args):
    from paper_2403_10616_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    if args.level_numel:
        cfg = cfg.scaled(tuple(args.level_numel for _ in cfg.level_numel),
                         name="%s-n%d" % (cfg.name, args.level_numel))
    return cfg


def time_steps(fn, steps, world):
    """K calls of fn between barrier + synchronize; returns (ms per step over the whole region,
    mean per-call ms from per-step event pairs)."""
    import torch
    stream = torch.cuda.current_stream()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier(world)
    torch.cuda.synchronize()
    for k in range(steps):
        starts[k].record(stream)
        fn()
        ends[k].record(stream)
    torch.cuda.synchronize()
    barrier(world)
    total = starts[0].elapsed_time(ends[-1])
    per_call = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    return total / steps, sum(per_call) / steps


def cpu_baseline_from_device(problem, sample_numel):
    """Oracle on a slab of the same workload: the first `sample_numel` parameters of every module
    and of every path's slot, copied back from the device."""
    import torch
    import oracle
    from paper_2403_10616_b200 import synth
    cfg = problem.cfg
    n = [min(sample_numel, x) for x in cfg.level_numel]
    small = cfg.scaled(n)
    mod_off = problem.module_offsets()
    lvl_off = problem.level_offsets()
    theta_parts, mom_parts = [], []
    for l, k in enumerate(cfg.modules_per_level):
        for e in range(k):
            src = int(mod_off[l]) + e * cfg.level_numel[l]
            theta_parts.append(problem.theta[src:src + n[l]])
            mom_parts.append(problem.momentum[src:src + n[l]])
    theta = torch.cat(theta_parts).cpu().numpy()
    momentum = torch.cat(mom_parts).cpu().numpy()
    paths = []
    for p in problem.paths:
        row = torch.cat([p[int(lvl_off[l]):int(lvl_off[l]) + n[l]] for l in range(cfg.num_levels)])
        row = row.cpu()
        if row.dtype == torch.bfloat16:
            paths.append(row.view(torch.int16).numpy().view(np.uint16))
        else:
            paths.append(row.numpy())
    threads = oracle.max_threads()
    dtype = oracle.BF16 if cfg.path_dtype == "bf16" else oracle.F32
    t0 = time.perf_counter()
    oracle.outer_sync(small.modules_per_level, small.level_numel, problem.table, theta, momentum,
                      paths, dtype, float(np.float32(cfg.outer_lr)),
                      float(np.float32(cfg.outer_momentum)), problem.weights, problem.reported,
                      threads)
    dt = time.perf_counter() - t0
    return {"value": small.path_params / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "seconds": dt,
            "sample": "one call on the first %s parameters of every level of all %d paths (%d "
                      "path-params), inputs copied back from the device" %
                      ("/".join(str(x) for x in n), cfg.num_paths, small.path_params)}


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the workload per step."""
    world, rank, _ = dist_setup(args)
    if rank != 0:
        return
    import oracle
    from paper_2403_10616_b200 import synth
    cfg = workload_config(args)
    n = [min(REF_SAMPLE_NUMEL, x) for x in cfg.level_numel]
    small = cfg.scaled(n)
    pr = synth.make_problem(small, "cpu")
    theta = pr.theta.numpy()
    momentum = pr.momentum.numpy()
    import torch
    if small.path_dtype == "bf16":
        paths = [p.view(torch.int16).numpy().view(np.uint16) for p in pr.paths]
    else:
        paths = [p.numpy() for p in pr.paths]
    threads = oracle.max_threads()
    dtype = oracle.BF16 if small.path_dtype == "bf16" else oracle.F32

    def step():
        oracle.outer_sync(small.modules_per_level, small.level_numel, pr.table, theta, momentum,
                          paths, dtype, float(np.float32(small.outer_lr)),
                          float(np.float32(small.outer_momentum)), pr.weights, pr.reported, threads)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = small.path_params / dt
    sample = ("each step: the oracle on %s parameters per level of all %d paths (%d path-params), "
              "synthetic inputs drawn on the host" % ("/".join(str(x) for x in n), small.num_paths,
                                                      small.path_params))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": cfg.name, "levels": list(cfg.modules_per_level),
                   "level_numel": list(cfg.level_numel), "paths": cfg.num_paths,
                   "path_dtype": cfg.path_dtype, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args):
    import torch
    from paper_2403_10616_b200 import binding as B
    from paper_2403_10616_b200 import synth

    world, rank, local = dist_setup(args)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the outer sync has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    B.load()

    cfg = workload_config(args)
    whole_cfg, whole_plan = cfg, None
    if args.mode == "sharded":
        # Section 3.3, sharded executor: rank r owns slab r of every module of the ONE workload and
        # holds only that slab of theta, momentum and of every path copy (compact layout).  The
        # slab is itself a grid with smaller modules; its synthetic values are drawn per rank.
        import dataclasses
        code_w = B.DIPACO_BF16 if cfg.path_dtype == "bf16" else B.DIPACO_F32
        whole_plan = B.dipaco_create(cfg.modules_per_level, cfg.level_numel,
                                     synth.path_table(cfg.modules_per_level), synth.path_weights(cfg),
                                     np.float32(cfg.outer_lr), np.float32(cfg.outer_momentum), code_w,
                                     0, device=-1)
        slabs = []
        for l in range(cfg.num_levels):
            a, b = B.dipaco_plan_shard(whole_plan, rank, world, l)
            slabs.append(b - a)
        cfg = dataclasses.replace(cfg.scaled(slabs, name="%s-shard%dof%d" % (cfg.name, rank, world)),
                                  seed=cfg.seed + rank)
    need = cfg.path_params * (2 if cfg.path_dtype == "bf16" else 4) + 8 * cfg.module_params
    free, _total = torch.cuda.mem_get_info(device)
    if need * 1.02 > free:
        raise SystemExit("workload needs %.1f GB of device memory, %.1f GB free" % (need / 1e9, free / 1e9))

    problem = synth.make_problem(cfg, device, separate_buffers=args.separate_buffers)
    torch.cuda.synchronize()
    ptrs = [p.data_ptr() for p in problem.paths]
    kernel = {"auto": B.DIPACO_KERNEL_AUTO, "vector": B.DIPACO_KERNEL_VECTOR,
              "scalar": B.DIPACO_KERNEL_SCALAR}[args.kernel]
    code = B.DIPACO_BF16 if cfg.path_dtype == "bf16" else B.DIPACO_F32

    def tune(ctx):
        B.dipaco_set_kernel(ctx, kernel)
        B.dipaco_set_tuning(ctx, args.ctas_per_sm, args.stages, args.units, args.io_slots)
        B.dipaco_set_work_items(ctx, args.item_kb * 1024, args.items_per_cta)
        return ctx

    def make_ctx(chunk_paths):
        return tune(B.dipaco_create(cfg.modules_per_level, cfg.level_numel, problem.table,
                                    problem.weights, np.float32(cfg.outer_lr),
                                    np.float32(cfg.outer_momentum), code, chunk_paths, local))

    # ---- resident one-pass mode: the headline value (--mode selects another leg for profiling)
    if args.mode == "sharded":
        ctx = tune(B.dipaco_create_shard(whole_plan, rank, world, local))
        B.dipaco_destroy(whole_plan)
    else:
        ctx = make_ctx(cfg.chunk_paths if args.mode == "chunked" else 0)
    second = None
    if args.mode == "adam":
        second = torch.zeros_like(problem.theta)
        B.dipaco_set_adam(ctx, second.data_ptr(), 0.9, 0.99, 1e-3, 0.0, 0)

    ptr_arr = B.ptr_array(ptrs)
    theta_ptr, momentum_ptr = problem.theta.data_ptr(), problem.momentum.data_ptr()
    stream_handle = int(torch.cuda.current_stream().cuda_stream)

    def step():
        B.dipaco_outer_sync(ctx, theta_ptr, momentum_ptr, ptr_arr, problem.reported, stream_handle)

    for _ in range(max(args.warmup, 0)):
        step()
    torch.cuda.synchronize()
    launches_before = B.dipaco_launch_count(ctx)
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ
                           else os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local])
    sampler.wait_first_sample()
    sampler.mark_start()
    ms_region, ms_call = time_steps(step, args.steps, world)
    sampler.mark_end()
    clocks = sampler.stop()
    launches = B.dipaco_launch_count(ctx) - launches_before
    status = B.dipaco_device_status(ctx)
    if status != B.DIPACO_OK:
        raise SystemExit("device status after the timed region: %s" % B.strerror(status))
    B.dipaco_destroy(ctx)

    ms_max, units_total = aggregate(ms_region, float(cfg.path_params), world, device)
    value = units_total / (ms_max * 1e-3)
    alg_bytes = synth.algorithmic_bytes(cfg, problem.reported)
    if args.mode == "adam":
        alg_bytes += 8 * cfg.module_params   # the second moment is read and written once
    del second
    peak, peak_kind = measured_peak_hbm()
    achieved = alg_bytes / (ms_call * 1e-3) / 1e9

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True,
        "scaling": "strong" if args.mode == "sharded" else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": whole_cfg.name, "levels": list(whole_cfg.modules_per_level),
            "level_numel": list(whole_cfg.level_numel), "paths": whole_cfg.num_paths,
            "path_dtype": whole_cfg.path_dtype,
            "mode": {"resident": "resident one-pass (all path copies in HBM)",
                     "chunked": "chunks of %d paths, partial sums carried (all chunks in HBM)" % cfg.chunk_paths,
                     "adam": "resident one-pass, Adam-family outer optimiser",
                     "sharded": "resident one-pass on this rank's slab of every module (compact "
                                "layout, no exchange between ranks)"}[args.mode],
            "l2": "inputs (%.1f GB per GPU) exceed L2, no flush between steps" % (need / 1e9),
            "parallelism": ("1 GPU" if world == 1 else
                            "one problem split over %d ranks by parameter slab, no collective" % world
                            if args.mode == "sharded" else "replicas only"),
            "kernel": args.kernel,
        },
        "clocks": clocks,
        "gpu_launches": int(launches),
        "effective_gbs": achieved,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak,
                     "traffic": (NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * alg_bytes
                                 if args.kernel == "auto" and cfg.name == "grid16x16" and args.mode == "resident"
                                 and sources_digest() == NCU_CAPTURE_SOURCES_SHA256 else None),
                     "traffic_from": NCU_CAPTURE_COMMAND,
                     "peak_kind": "of " + peak_kind,
                     "kernel": "sync_bulk_kernel" if args.kernel == "auto" else "sync_direct_kernel",
                     "algorithmic_bytes_per_launch": alg_bytes, "ms_per_launch": ms_call,
                     "frac_of_nominal_8tbs": achieved / 8000.0},
    }

    # ---- the same launch with the optional features switched on (resident mode, rank 0)
    if not args.no_variants and rank == 0 and args.mode != "sharded":
        result["variants"] = run_variants(args, cfg, problem, make_ctx, ptrs, alg_bytes)

    # ---- the same workload walked in chunks of paths (device resident)
    if not args.no_chunked and cfg.chunk_paths > 0 and rank == 0 and args.mode != "sharded":
        ctx = make_ctx(cfg.chunk_paths)
        chunk_step = lambda: B.dipaco_outer_sync(ctx, theta_ptr, momentum_ptr, ptr_arr, problem.reported,
                                                 stream_handle)
        for _ in range(max(args.warmup, 1)):
            chunk_step()
        before = B.dipaco_launch_count(ctx)
        ms_c, _ = time_steps(chunk_step, args.steps, 1)
        moved, n_launch = B.dipaco_plan_traffic(ctx, problem.reported)
        result["chunked"] = {"chunk_paths": cfg.chunk_paths, "ms_per_step": ms_c,
                             "bytes_moved_by_construction": moved,
                             "moved_gbs": moved / (ms_c * 1e-3) / 1e9,
                             "frac_of_peak": moved / (ms_c * 1e-3) / 1e9 / peak,
                             "value": cfg.path_params / (ms_c * 1e-3), "unit": UNIT,
                             "effective_gbs": alg_bytes / (ms_c * 1e-3) / 1e9,
                             "gpu_launches": int(B.dipaco_launch_count(ctx) - before)}
        # the same walk through the chunk API, as a caller that holds one chunk at a time drives
        # it: accumulate every chunk in order, then a write-back launch per chunk
        nchunks, _ = B.dipaco_plan_chunks(ctx)
        cp = cfg.chunk_paths
        chunk_arrs = [B.ptr_array(ptrs[c * cp:(c + 1) * cp]) for c in range(nchunks)]

        def api_step():
            B.dipaco_sync_begin(ctx, theta_ptr, momentum_ptr, problem.reported, stream_handle)
            for c in range(nchunks):
                B.dipaco_sync_accumulate(ctx, c, chunk_arrs[c])
            for c in range(nchunks):
                B.dipaco_sync_writeback(ctx, c, chunk_arrs[c])
            B.dipaco_sync_end(ctx)

        try:
            api_step()
            before = B.dipaco_launch_count(ctx)
            api_steps = max(3, min(args.steps, 8))
            ms_api, _ = time_steps(api_step, api_steps, 1)
            result["chunked"]["chunk_api"] = {
                "ms_per_step": ms_api, "steps": api_steps,
                "gpu_launches": int(B.dipaco_launch_count(ctx) - before),
                "note": "dipaco_sync_begin / accumulate x%d / writeback x%d / end over the same "
                        "buffers; write-back launches read the bf16 cast scratch" % (nchunks, nchunks)}
        except B.DipacoError as exc:
            result["chunked"]["chunk_api"] = {"error": str(exc)}
        B.dipaco_destroy(ctx)

    # ---- CPU oracle on a slab of the same inputs (rank 0, N = 1)
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        result["cpu_baseline"] = cpu_baseline_from_device(problem, CPU_SAMPLE_NUMEL)

    # ---- end to end through the host-buffer entry point
    if not args.no_e2e:
        result["e2e"] = run_e2e(args, cfg, problem, make_ctx, world, device)

    # ---- the other workloads of the method's evaluation, same kernel and defaults (N = 1 only:
    # with more ranks the other GPUs would idle meanwhile)
    if not args.no_other_workloads and world == 1 and args.mode == "resident" and not args.level_numel:
        problem.paths.clear()
        problem.storage = None
        problem.theta = problem.momentum = None
        torch.cuda.empty_cache()
        result["other_workloads"] = run_other_workloads(args, cfg.name, tune, local, peak)

    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_variants(args, cfg, problem, make_ctx, ptrs, alg_bytes):
    """ms per synchronisation with the optional features on: gradient rescaling by sqrt(paths per
    module), heavy-ball and SGD outer optimisers, and the Adam family (one more fp32 state array:
    8 more bytes per module parameter)."""
    import torch
    from paper_2403_10616_b200 import binding as B
    steps = max(3, min(args.steps, 8))
    out = {}

    def timed(ctx):
        fn = lambda: B.dipaco_outer_sync(ctx, problem.theta.data_ptr(), problem.momentum.data_ptr(),
                                         ptrs, problem.reported)
        for _ in range(2):
            fn()
        ms, _ = time_steps(fn, steps, 1)
        ok = B.dipaco_device_status(ctx) == B.DIPACO_OK
        B.dipaco_destroy(ctx)
        return ms if ok else None

    ctx = make_ctx(0)
    scale = np.concatenate([np.full(k, np.sqrt(cfg.num_paths / k), dtype=np.float32)
                            for k in cfg.modules_per_level])
    B.dipaco_set_module_scale(ctx, scale)
    out["rescaled_sqrt_paths_ms"] = timed(ctx)
    for name, opt in (("heavy_ball_ms", B.DIPACO_OPT_MOMENTUM), ("sgd_ms", B.DIPACO_OPT_SGD)):
        ctx = make_ctx(0)
        B.dipaco_set_optimizer(ctx, opt)
        out[name] = timed(ctx)
    try:
        second = torch.zeros_like(problem.theta)
    except RuntimeError:
        second = None
    if second is not None:
        ctx = make_ctx(0)
        B.dipaco_set_adam(ctx, second.data_ptr(), 0.9, 0.99, 1e-3, 0.0, 0)
        ms = timed(ctx)
        out["adam_ms"] = ms
        if ms:
            out["adam_gbs"] = (alg_bytes + 8 * cfg.module_params) / (ms * 1e-3) / 1e9
        del second
        torch.cuda.empty_cache()
    out["steps"] = steps
    return out


def run_other_workloads(args, skip_name, tune, local, peak):
    """ms per synchronisation of the remaining workloads (resident one-pass, default kernel).  Each
    timed region lasts at least 0.6 s so that the clock sampler sees it; the 2x2 grid (9 MB, L2
    resident) is a latency figure, reported in microseconds per call."""
    import math
    import torch
    from paper_2403_10616_b200 import binding as B
    from paper_2403_10616_b200 import synth
    out = []
    # the last entry is the 16x16 grid with an odd level size: every module of theta and every slot
    # of every path copy then starts inside a 16-byte unit (rows of one block: all eight positions),
    # so the bulk-copy kernel cannot take it and the shifted vector kernel does
    odd = synth.CONFIGS["grid16x16-odd-level-size"]
    for name in ("grid2x2", "grid4x4", "grid16x16-masked", "grid4x4x4x4", odd.name):
        if name == skip_name:
            continue
        cfg = odd if name == odd.name else synth.CONFIGS[name]
        es = 2 if cfg.path_dtype == "bf16" else 4
        need = cfg.path_params * es + 8 * cfg.module_params
        torch.cuda.empty_cache()
        free, _ = torch.cuda.mem_get_info()
        if need * 1.02 > free:
            out.append({"workload": name, "skipped": "needs %.1f GB, %.1f GB free" % (need / 1e9, free / 1e9)})
            continue
        problem = synth.make_problem(cfg, "cuda:%d" % local)
        code = B.DIPACO_BF16 if cfg.path_dtype == "bf16" else B.DIPACO_F32
        ctx = tune(B.dipaco_create(cfg.modules_per_level, cfg.level_numel, problem.table, problem.weights,
                                   np.float32(cfg.outer_lr), np.float32(cfg.outer_momentum), code, 0, local))
        arr = B.ptr_array([p.data_ptr() for p in problem.paths])
        th, mo = problem.theta.data_ptr(), problem.momentum.data_ptr()
        handle = int(torch.cuda.current_stream().cuda_stream)
        fn = lambda: B.dipaco_outer_sync(ctx, th, mo, arr, problem.reported, handle)
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(10):
            fn()
        b.record()
        torch.cuda.synchronize()
        probe_ms = max(a.elapsed_time(b) / 10, 1e-3)
        steps = int(min(max(math.ceil(600.0 / probe_ms), 20), 200000))
        sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ
                               else os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local])
        sampler.wait_first_sample()
        torch.cuda.synchronize()
        sampler.mark_start()
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        sampler.mark_end()
        clocks = sampler.stop()
        ms = a.elapsed_time(b) / steps
        graph_us = None
        if need < 126e6:
            # launch-bound: the same repeated call (it reuses the kept plan, so it only launches)
            # captured 100 times in a CUDA graph and replayed
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                h = int(torch.cuda.current_stream().cuda_stream)
                for _ in range(100):
                    B.dipaco_outer_sync(ctx, th, mo, arr, problem.reported, h)
            replays = max(steps // 100, 10)
            graph.replay()
            torch.cuda.synchronize()
            a.record()
            for _ in range(replays):
                graph.replay()
            b.record()
            torch.cuda.synchronize()
            graph_us = a.elapsed_time(b) / (replays * 100) * 1e3
            del graph
        ok = B.dipaco_device_status(ctx) == B.DIPACO_OK
        B.dipaco_destroy(ctx)
        alg = synth.algorithmic_bytes(cfg, problem.reported)
        entry = {"workload": name, "steps": steps, "ms_per_step": ms, "status_ok": ok,
                 "value": cfg.path_params / (ms * 1e-3), "unit": UNIT,
                 "algorithmic_bytes": alg, "clocks": clocks}
        if need < 126e6:
            entry["us_per_call"] = ms * 1e3
            entry["us_per_call_cuda_graph"] = graph_us
            entry["note"] = "fits in L2: launch latency, not a roofline point"
        else:
            gbs = alg / (ms * 1e-3) / 1e9
            entry.update({"algorithmic_gbs": gbs, "frac_of_peak": gbs / peak,
                          "frac_of_nominal_8tbs": gbs / 8000.0})
            if name == odd.name:
                entry["level_numel"] = list(cfg.level_numel)
                entry["kernel"] = "sync_direct_kernel<.,8,shifted> (buffers at odd element offsets)"
        out.append(entry)
        del problem, arr
        torch.cuda.empty_cache()
    return out


def host_memory_available():
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return None


def run_e2e(args, cfg, problem, make_ctx, world, device):
    """Same metric through dipaco_outer_sync_host: state in pinned host memory, every step copies
    the inputs host->device and the results device->host inside the timed region.  When the host
    cannot pin one full copy of the workload per rank, the leg runs on the first n parameters of
    every level (same grid, same paths) and says so."""
    import torch
    from paper_2403_10616_b200 import binding as B
    chunk = cfg.chunk_paths if cfg.chunk_paths > 0 else min(32, cfg.num_paths)
    es = 2 if cfg.path_dtype == "bf16" else 4
    local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
    full_bytes = cfg.path_params * es + 8 * cfg.module_params
    avail = host_memory_available()
    numel = list(cfg.level_numel)
    note = None
    if avail is not None and full_bytes * 1.15 > 0.8 * avail / max(local_world, 1):
        frac = (0.8 * avail / max(local_world, 1)) / (full_bytes * 1.15)
        numel = [max(8192, int(n * frac) // 8192 * 8192) for n in cfg.level_numel]
        note = ("host memory (%.0f GB available, %d ranks) does not hold the full workload: run on "
                "the first %s parameters of every level" % (avail / 1e9, local_world,
                                                             "/".join(str(n) for n in numel)))
    small = cfg if note is None else cfg.scaled(numel)
    mod_off = problem.module_offsets()
    lvl_off = problem.level_offsets()
    try:
        theta_h = torch.empty(small.module_params, dtype=torch.float32, pin_memory=True)
        mom_h = torch.empty(small.module_params, dtype=torch.float32, pin_memory=True)
        paths_h = torch.empty((small.num_paths, small.params_per_path), dtype=problem.paths[0].dtype,
                              pin_memory=True)
    except RuntimeError as exc:
        return {"value": None, "unit": UNIT, "error": "could not pin host memory: %s" % exc}
    pcie = pcie_probe(paths_h, device)
    dst = 0
    for l, k in enumerate(cfg.modules_per_level):
        for e in range(k):
            src = int(mod_off[l]) + e * cfg.level_numel[l]
            theta_h[dst:dst + numel[l]].copy_(problem.theta[src:src + numel[l]])
            mom_h[dst:dst + numel[l]].copy_(problem.momentum[src:src + numel[l]])
            dst += numel[l]
    for i, p in enumerate(problem.paths):
        dst = 0
        for l in range(cfg.num_levels):
            paths_h[i, dst:dst + numel[l]].copy_(p[int(lvl_off[l]):int(lvl_off[l]) + numel[l]])
            dst += numel[l]
    torch.cuda.synchronize()
    # the device copies are no longer needed: free them so the staging buffers fit
    problem.paths.clear()
    problem.storage = None
    torch.cuda.empty_cache()
    code = B.DIPACO_BF16 if small.path_dtype == "bf16" else B.DIPACO_F32
    ctx = B.dipaco_create(small.modules_per_level, small.level_numel, problem.table, problem.weights,
                          np.float32(small.outer_lr), np.float32(small.outer_momentum), code, chunk,
                          device.index)
    hptrs = [paths_h[i].data_ptr() for i in range(small.num_paths)]

    def step():
        B.dipaco_outer_sync_host(ctx, theta_h.data_ptr(), mom_h.data_ptr(), hptrs, problem.reported)

    if args.host_unit_mb:
        B.dipaco_set_host_unit_bytes(ctx, args.host_unit_mb << 20)
    B.dipaco_set_host_threads(ctx, args.host_threads)
    step()   # warm-up: allocates the staging buffers
    steps = max(1, args.e2e_steps)
    barrier(world)
    torch.cuda.synchronize()
    per_step = []
    t0 = time.perf_counter()
    for _ in range(steps):
        t1 = time.perf_counter()
        step()          # synchronous: returns when the host buffers hold the result
        per_step.append((time.perf_counter() - t1) * 1e3)
    torch.cuda.synchronize()
    dt_ms = (time.perf_counter() - t0) * 1e3 / steps
    barrier(world)
    ms_max, units = aggregate(dt_ms, float(small.path_params), world, device)
    n_rep = small.num_paths if problem.reported is None else int(problem.reported.sum())
    B.dipaco_destroy(ctx)
    results_bytes = 8 * small.module_params + small.num_paths * small.params_per_path * es
    if args.host_threads != 0:
        # the new value of a module crosses PCIe once; host threads copy it into every path
        d2h = (8 + es) * small.module_params
    else:
        d2h = results_bytes
    out = {"value": units / (ms_max * 1e-3), "unit": UNIT, "ms_per_step": ms_max, "steps": steps,
           "ms_per_step_min": min(per_step), "ms_per_step_mean": sum(per_step) / len(per_step),
           "h2d_bytes_per_step": 8 * small.module_params + n_rep * small.params_per_path * es,
           "d2h_bytes_per_step": d2h,
           "host_result_bytes_per_step": results_bytes,
           "api": "dipaco_outer_sync_host, pinned host buffers, slab-ordered streaming, staging "
                  "bounded by %d path copies; %s" % (
                      chunk, "every path copy downloaded" if args.host_threads == 0 else
                      "each module's new value downloaded once and copied into its paths by host threads")}
    if pcie:
        # what this box's PCIe link gives a plain pinned copy, measured in this process: the
        # step cannot be faster than the bytes of the busier direction at the both-ways rate
        # (both directions equally loaded: the both-ways rate; otherwise each at its one-way rate)
        if out["d2h_bytes_per_step"] >= 0.8 * out["h2d_bytes_per_step"]:
            busier = max(out["h2d_bytes_per_step"], out["d2h_bytes_per_step"])
            ideal_ms = busier / (pcie["both_ways_each_gbs"] * 1e9) * 1e3
        else:
            ideal_ms = max(out["h2d_bytes_per_step"] / pcie["h2d_gbs"],
                           out["d2h_bytes_per_step"] / pcie["d2h_gbs"]) / 1e9 * 1e3
        pcie["ideal_ms_per_step"] = ideal_ms
        pcie["frac_of_ideal"] = ideal_ms / ms_max
        out["pcie"] = pcie
    if note:
        out["reduced"] = note
    return out


def pcie_probe(pinned, device, nbytes=2 << 30, reps=3):
    """GB/s of plain pinned copies on this machine: host->device alone, device->host alone and both at
    once (per direction), on 2 GiB pieces of the (not yet filled) pinned block of the end-to-end leg."""
    import torch
    flat = pinned.view(-1).view(torch.uint8)
    if flat.numel() < 2 * nbytes:
        return None
    try:
        dev_in = torch.empty(nbytes, dtype=torch.uint8, device=device)
        dev_out = torch.zeros(nbytes, dtype=torch.uint8, device=device)
    except RuntimeError:
        return None
    up, down = torch.cuda.Stream(device), torch.cuda.Stream(device)

    def run(do_up, do_down):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(reps):
            if do_up:
                with torch.cuda.stream(up):
                    dev_in.copy_(flat[:nbytes], non_blocking=True)
            if do_down:
                with torch.cuda.stream(down):
                    flat[nbytes:2 * nbytes].copy_(dev_out, non_blocking=True)
        torch.cuda.synchronize()
        return nbytes * reps / (time.perf_counter() - t0) / 1e9

    run(True, True)
    out = {"h2d_gbs": run(True, False), "d2h_gbs": run(False, True), "both_ways_each_gbs": run(True, True)}
    del dev_in, dev_out
    torch.cuda.empty_cache()
    return out


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
