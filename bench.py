#!/usr/bin/env python
"""Benchmark of the N-way Adasum combine.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

A step is one whole reduce (every level: partial Gram matrices, tree weights, weighted sum) of one
synthetic workload.  Prints ONE JSON line.  `value` is input GB/s (N_workers * elements * bytes
per element / time per reduce) with the inputs resident in device memory; `e2e` is the same metric
with the inputs starting in pinned host memory and the result ending there.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2006_02924_b200 import workloads  # noqa: E402

METRIC = "adasum_nway_reduce_input_throughput"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures of the
# kernels as built from the source whose fingerprint is recorded with them; see profiles/.
# {(workload, kernel, level): bytes}.  Reported only while the kernel source is unchanged.
NCU_TRAFFIC = {
    "fingerprint": "c99f9f3e55777864",
    "bytes": {
        "c2/gram_partial/0": 822090496,      # profiles/gram_partial_mma_f32_r8_c2.txt
        "c2/weighted_sum/0": 874237696,      # profiles/weighted_sum_f32_r8_c2.txt
        "c1/fused_small/0": 8040448,         # profiles/fused_small_f32_r2_c1.txt
    },
}


def kernel_source_fingerprint() -> str:
    import hashlib

    h = hashlib.sha256()
    for name in ("adasum_kernels.cuh", "adasum_f64.cuh", "adasum_api.cu"):
        with open(os.path.join(ROOT, "paper_2006_02924_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---- clocks -----------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._handle = None
        try:
            import pynvml

            self.nvml = pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(device_index)
            handle = None
            uuid = getattr(props, "uuid", None)
            if uuid is not None:
                try:
                    handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    handle = None
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._handle = handle
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception as exc:  # NVML missing: report that instead of inventing numbers
            self.error = repr(exc)

    def sample_once(self):
        if self._handle is None:
            return
        try:
            mhz = int(self.nvml.nvmlDeviceGetClockInfo(self._handle, self.nvml.NVML_CLOCK_SM))
            try:
                mask = int(self.nvml.nvmlDeviceGetCurrentClocksEventReasons(self._handle))
            except Exception:
                mask = int(self.nvml.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle))
            self.samples.append(mhz)
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_once()
            self._stop.wait(self.period)

    def __enter__(self):
        self._stop.clear()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self.sample_once()
        self._stop.set()
        self._thread.join()

    def summary(self) -> dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                    "samples": 0, "error": getattr(self, "error", "no samples")}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---- the CUDA arm ------------------------------------------------------------------------------------

def algorithmic_bytes(record, plan_levels, total_elems, in_bytes):
    """Bytes one launch must move: its operands once, plus its output for the weighted sum."""
    level = plan_levels[record["level"]]
    elem_bytes = in_bytes if record["level"] == 0 else 4
    read = level["operands"] * total_elems * elem_bytes
    if record["kernel"] == "gram_partial":
        return read
    if record["kernel"] == "weighted_sum":
        return read + level["groups"] * total_elems * 4
    if record["kernel"] == "fused_small":      # both passes in one launch: HBM sees the operands once
        return read + total_elems * 4
    if record["kernel"] == "wsum_gram":        # pass 2 of this level and pass 1 of the next from the same registers
        return read + level["groups"] * total_elems * 4
    if record["kernel"] == "convert":
        return total_elems * (in_bytes + 4)
    return 0


def plan_levels_of(lib, wl, flags):
    info = lib.adasum_plan_info(wl.total_elems, wl.num_tensors, wl.n_workers, wl.spec.dtype, flags)
    levels, m = [], wl.n_workers
    for r in info["radices"]:
        g = (m + r - 1) // r
        levels.append({"radix": r, "operands": m, "groups": g})
        m = g
    return info, levels


L2_FLUSH_BYTES = 512 * 1024 * 1024      # four times the 126 MB L2


def time_reduce(lib, wl, steps, warmup, flags, world=1, sampler=None, flush=True):
    """W warm-up steps, then K timed steps bracketed by barrier + synchronize.  Every step is timed
    with its own pair of CUDA events on the launching stream; between steps a buffer four times the
    size of L2 is overwritten (outside the events), so no step finds its inputs cached by the
    previous one.  Returns ms per step (local): the mean of the K event intervals."""
    import torch.distributed as dist

    dev = wl.grads[0].device
    out = torch.empty(wl.total_elems, dtype=torch.float32, device=dev)
    need = lib.adasum_workspace_bytes(wl.total_elems, wl.num_tensors, wl.n_workers, wl.spec.dtype, flags)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    scrub = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev) if flush else None
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        lib.adasum_reduce(wl.grads, wl.offsets, out=out, workspace=ws, flags=flags, stream=stream)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ctx = sampler if sampler is not None else _Null()
    with ctx:
        for i in range(steps):
            if scrub is not None:
                scrub.zero_()
            starts[i].record(stream)
            lib.adasum_reduce(wl.grads, wl.offsets, out=out, workspace=ws, flags=flags, stream=stream)
            stops[i].record(stream)
        if sampler is not None:
            sampler.sample_once()
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = sum(a.elapsed_time(b) for a, b in zip(starts, stops)) / steps
    return ms, out, ws


def time_variants(lib, wl, steps, warmup, flags):
    """The same workload through adasum_reduce_delta: with a start buffer (the optimizer-delta form,
    result written over the start buffer) and with bf16 output.  Per-step events, L2 flushed."""
    dev = wl.grads[0].device
    dt = wl.grads[0].dtype
    need = lib.adasum_workspace_bytes(wl.total_elems, wl.num_tensors, wl.n_workers, wl.spec.dtype, flags)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    scrub = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    gen = torch.Generator(device=dev)
    gen.manual_seed(workloads.BASE_SEED + 99)
    params = torch.randn(wl.total_elems, generator=gen, device=dev).to(dt)
    out16 = torch.empty(wl.total_elems, dtype=torch.bfloat16, device=dev)
    b = workloads.DTYPE_BYTES[wl.spec.dtype]
    cases = [
        ("delta form, parameters updated in place",
         lambda: lib.adasum_reduce_delta(wl.grads, params, wl.offsets, out=params, workspace=ws, flags=flags,
                                         stream=stream),
         2 * (wl.n_workers + 1) * wl.total_elems * b + wl.total_elems * b),
        ("plain reduce, bf16 output",
         lambda: lib.adasum_reduce_delta(wl.grads, None, wl.offsets, out=out16, workspace=ws, flags=flags,
                                         stream=stream),
         2 * wl.n_workers * wl.total_elems * b + 2 * wl.total_elems),
    ]
    if wl.spec.dtype == "f32" and wl.input_bytes <= 4e9:
        # the same values as fp64 buffers: the fp64 kernels (levels of radix 4 / 2, doubles throughout)
        grads64 = [g.double() for g in wl.grads]
        out64 = torch.empty(wl.total_elems, dtype=torch.float64, device=dev)
        info64 = lib.adasum_plan_info(wl.total_elems, wl.num_tensors, wl.n_workers, "f64", 0)
        ws64 = torch.empty(max(lib.adasum_workspace_bytes(wl.total_elems, wl.num_tensors, wl.n_workers, "f64", 0), 256),
                           dtype=torch.uint8, device=dev)
        moved, m = 0, wl.n_workers
        for r in info64["radices"]:             # every level: operands read twice, outputs written once
            g = (m + r - 1) // r
            moved += (2 * m + g) * wl.total_elems * 8
            m = g
        cases.append((f"fp64 buffers, fp64 output, radices {info64['radices']}",
                      lambda: lib.adasum_reduce_delta(grads64, None, wl.offsets, out=out64, workspace=ws64,
                                                      stream=stream), moved))
    results = []
    for name, call, two_read_bytes in cases:
        for _ in range(warmup):
            call()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        torch.cuda.synchronize()
        for i in range(steps):
            scrub.zero_()
            starts[i].record(stream)
            call()
            stops[i].record(stream)
        torch.cuda.synchronize()
        ms = sum(a.elapsed_time(c) for a, c in zip(starts, stops)) / steps
        in_bytes = wl.input_bytes * (2 if name.startswith("fp64") else 1)
        results.append({"variant": name, "ms_per_reduce": ms, "input_gbs": in_bytes / (ms * 1e-3) / 1e9,
                        "two_read_bytes": two_read_bytes,
                        "two_read_gbs": two_read_bytes / (ms * 1e-3) / 1e9})
    return results


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


def kernel_breakdown(lib, wl, steps, flags, out, ws):
    """The same K steps again with an event after every launch; per (kernel, level): launches,
    mean ms, total ms."""
    info, levels = plan_levels_of(lib, wl, flags)
    stream = torch.cuda.current_stream()
    lib.adasum_profile_enable(steps * max(info["launches"], 1) + 8)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    scrub = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=out.device)
    t0.record(stream)
    for _ in range(steps):
        scrub.zero_()
        lib.adasum_reduce(wl.grads, wl.offsets, out=out, workspace=ws, flags=flags, stream=stream)
    t1.record(stream)
    torch.cuda.synchronize()
    del scrub
    records = lib.adasum_profile_collect(steps * max(info["launches"], 1) + 8)
    groups = {}
    for r in records:
        key = (r["kernel"], r["level"])
        g = groups.setdefault(key, {"kernel": r["kernel"], "level": r["level"], "radix": r["radix"],
                                    "launches": 0, "total_ms": 0.0})
        g["launches"] += 1
        g["total_ms"] += r["ms"]
    rows = []
    in_bytes = workloads.DTYPE_BYTES[wl.spec.dtype]
    for g in groups.values():
        g["mean_ms"] = g["total_ms"] / g["launches"]
        g["bytes_per_launch"] = algorithmic_bytes(g, levels, wl.total_elems, in_bytes)
        g["gbs"] = g["bytes_per_launch"] / (g["mean_ms"] * 1e-3) / 1e9 if g["mean_ms"] > 0 else 0.0
        rows.append(g)
    rows.sort(key=lambda g: -g["total_ms"])
    return rows, sum(g["total_ms"] for g in rows) / steps, info, levels


def time_e2e(lib, wl, steps, flags, out, ws):
    """Inputs start in pinned host memory every step and the result is read back to the host."""
    dev = wl.grads[0].device
    host_in = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True).copy_(g) for g in wl.grads]
    host_out = torch.empty(wl.total_elems, dtype=torch.float32, pin_memory=True)
    staging = [torch.empty_like(g) for g in wl.grads]
    stream = torch.cuda.current_stream()

    def step():
        for d, h in zip(staging, host_in):
            d.copy_(h, non_blocking=True)
        lib.adasum_reduce(staging, wl.offsets, out=out, workspace=ws, flags=flags, stream=stream)
        host_out.copy_(out, non_blocking=True)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.perf_counter()
    t0.record(stream)
    for _ in range(steps):
        step()
    t1.record(stream)
    torch.cuda.synchronize()
    wall = (time.perf_counter() - wall0) * 1e3 / steps
    ms = max(t0.elapsed_time(t1) / steps, wall)
    del dev
    return ms, wl.input_bytes, wl.total_elems * 4, float(host_out[:8].abs().sum())


# ---- the CPU oracle arm ------------------------------------------------------------------------------

def oracle_sample(wl_cpu, budget_elem_ops: float):
    """A prefix-free sample of whole tensors (largest first until the budget is used) whose
    reduction costs about budget_elem_ops = 2 (N-1) * elements."""
    sizes = np.diff(wl_cpu.offsets)
    per_elem = 2.0 * max(wl_cpu.n_workers - 1, 1)
    order = np.argsort(-sizes, kind="stable")
    chosen, used = [], 0.0
    for t in order:
        cost = per_elem * float(sizes[t])
        if chosen and used + cost > budget_elem_ops:
            continue
        chosen.append(int(t))
        used += cost
        if used >= budget_elem_ops:
            break
    chosen.sort()
    return chosen


def run_oracle(wl, tensors, threads=0):
    """Times the fp64 oracle, as it stands, on the chosen tensors.  Returns (seconds, input bytes,
    threads used)."""
    from oracle import adasum_oracle as oracle

    dtype = wl.spec.dtype
    pieces, sizes = [], []
    for t in tensors:
        lo, hi = int(wl.offsets[t]), int(wl.offsets[t + 1])
        pieces.append((lo, hi))
        sizes.append(hi - lo)
    offs = workloads.offsets_from_sizes(sizes)
    host = []
    for g in wl.grads:
        cat = torch.cat([g[lo:hi] for lo, hi in pieces]).cpu().contiguous()
        host.append(cat.view(torch.uint16).numpy() if dtype == "bf16" else cat.numpy())
    oracle.build()
    used = oracle.threads_used(threads)
    t0 = time.perf_counter()
    oracle.adasum_reduce(host, offsets=offs, dtype=dtype, threads=threads)
    dt = time.perf_counter() - t0
    nbytes = len(host) * int(offs[-1]) * workloads.DTYPE_BYTES[dtype]
    return dt, nbytes, used


def reference_arm(args):
    """`--impl reference`: the CPU oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = workloads.SPECS[args.workload]
    steps, warmup = max(args.steps, 1), max(args.warmup, 0)
    # keep host memory and generation time bounded: materialise at most 2.5e8 input elements
    sizes = spec.tensor_sizes()
    cap = 250_000_000 // spec.n_workers
    keep, acc = [], 0
    for t in np.argsort(-np.asarray(sizes), kind="stable"):
        if acc + sizes[t] <= cap:
            keep.append(int(t))
            acc += sizes[t]
    keep.sort()
    wl = workloads.generate(spec, device="cpu", tensor_sizes=[sizes[t] for t in keep])
    all_tensors = list(range(wl.num_tensors))
    # calibrate on a small sample, then size each step so that the whole run stays near two minutes
    probe = oracle_sample(wl, 2e8)
    dt, nbytes, threads = run_oracle(wl, probe)
    per_elem = 2.0 * max(spec.n_workers - 1, 1)
    probe_ops = per_elem * sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in probe)
    rate = probe_ops / max(dt, 1e-6)
    budget = rate * min(120.0 / (steps + warmup), 20.0)
    full_ops = per_elem * wl.total_elems
    tensors = all_tensors if budget >= full_ops else oracle_sample(wl, budget)
    times = []
    for i in range(steps + warmup):
        dt, nbytes, threads = run_oracle(wl, tensors)
        if i >= warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = nbytes / (ms * 1e-3) / 1e9
    sample = (f"{len(tensors)} of {len(sizes)} tensors of {args.workload} "
              f"({sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in tensors)} elements x {spec.n_workers} workers)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "n_workers": spec.n_workers, "input_dtype": spec.dtype,
                   "tensor_list": spec.tensor_list, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---- main ---------------------------------------------------------------------------------------------

def aggregate_over_ranks(ms_local: float, bytes_local: float, world: int, device="cpu"):
    """Whole-job figures of a run with one independent workload per rank: the step time is the
    slowest rank's, the work is the sum over ranks.  Returns (ms, total bytes)."""
    if world <= 1:
        return ms_local, bytes_local
    import torch.distributed as dist

    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    b = torch.tensor([bytes_local], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), float(b.item())


def resolve_spec(name, n_workers=None, tensor_list=None):
    """The named configuration, optionally with another worker count / tensor list (smaller cases
    of the same kernels, e.g. for profiler captures)."""
    import dataclasses

    spec = workloads.SPECS[name]
    if n_workers:
        spec = dataclasses.replace(spec, n_workers=int(n_workers))
    if tensor_list:
        spec = dataclasses.replace(spec, tensor_list=tensor_list)
    return spec


def measure_workload(lib, name, steps, warmup, flags, replica, world, sampler=None):
    wl = workloads.generate(name, device="cuda", replica=replica)
    ms, out, ws = time_reduce(lib, wl, steps, warmup, flags, world=world, sampler=sampler)
    return wl, ms, out, ws


def summarise(wl, ms, peak):
    p, b, n = wl.total_elems, workloads.DTYPE_BYTES[wl.spec.dtype], wl.n_workers
    one_read = n * p * b + 4 * p
    return {
        "ms_per_reduce": ms,
        "input_gbs": wl.input_bytes / (ms * 1e-3) / 1e9,
        "one_read_roofline_frac_measured_peak": one_read / (ms * 1e-3) / 1e9 / peak,
        "one_read_roofline_frac_nominal_8TBs": one_read / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "two_read_roofline_frac_measured_peak": (2 * n * p * b + 4 * p) / (ms * 1e-3) / 1e9 / peak,
    }


def cuda_arm(args):
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2006_02924_b200 import binding as lib

    flags = lib.flags_radix(args.radix_first, args.radix_later)
    if args.no_level_fusion:
        flags |= lib.ADASUM_FLAG_NO_LEVEL_FUSION
    if args.no_tcgen05:
        flags |= lib.ADASUM_FLAG_NO_TCGEN05
    peak, peak_kind = measured_peak()
    sampler = ClockSampler(local_rank)
    steps, warmup = max(args.steps, 1), max(args.warmup, 3)

    main_spec = resolve_spec(args.workload, args.n_workers, args.tensor_list)
    wl, ms_local, out, ws = measure_workload(lib, main_spec, steps, warmup, flags, rank, world, sampler)
    ms, job_bytes = aggregate_over_ranks(ms_local, float(wl.input_bytes), world, "cuda")
    value = job_bytes / (ms * 1e-3) / 1e9

    rows, ms_instrumented, info, levels = kernel_breakdown(lib, wl, steps, flags, out, ws)
    top = rows[0]
    traffic = None
    if NCU_TRAFFIC["fingerprint"] == kernel_source_fingerprint():
        traffic = NCU_TRAFFIC["bytes"].get(f"{args.workload}/{top['kernel']}/{top['level']}")
    roofline = {
        "bound": "hbm", "kernel": f"{top['kernel']}<radix {top['radix']}> level {top['level']}",
        "achieved": top["gbs"], "peak": peak, "unit": "GB/s", "frac": top["gbs"] / peak,
        "peak_kind": f"of {peak_kind}", "traffic": traffic,
        "bytes_per_launch": top["bytes_per_launch"], "mean_launch_ms": top["mean_ms"],
        "share_of_step": top["total_ms"] / sum(r["total_ms"] for r in rows),
        "timing": "CUDA event after every launch, same K steps (L2 flushed between them) repeated right "
                  "after the timed region",
        "instrumented_ms_per_step": ms_instrumented,
        "kernels": [{k: r[k] for k in ("kernel", "level", "radix", "launches", "mean_ms", "gbs")} for r in rows],
    }

    e2e_steps = min(steps, 20)
    e2e_ms_local, h2d, d2h, _ = time_e2e(lib, wl, e2e_steps, flags, out, ws)
    e2e_ms, _ = aggregate_over_ranks(e2e_ms_local, float(wl.input_bytes), world, "cuda")
    e2e = {"value": job_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        budget = 4e9
        tensors = oracle_sample(wl, budget)
        if 2.0 * (wl.n_workers - 1) * wl.total_elems <= budget:
            tensors = list(range(wl.num_tensors))
        dt, nbytes, threads = run_oracle(wl, tensors)
        cpu_baseline = {
            "value": nbytes / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{len(tensors)} of {wl.num_tensors} tensors of {args.workload}, "
                      f"{sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in tensors)} elements x "
                      f"{wl.n_workers} workers, {dt:.2f} s",
        }

    summary = summarise(wl, ms, peak)
    spec = wl.spec
    n_workers, total_elems, num_tensors = wl.n_workers, wl.total_elems, wl.num_tensors
    del out, ws
    variants = []
    if rank == 0 and world == 1 and not args.no_other_workloads:
        variants = time_variants(lib, wl, max(3, min(steps, 200)), 3, flags)
    del wl
    torch.cuda.empty_cache()

    others = []
    if rank == 0 and world == 1 and not args.no_other_workloads:
        for name in ("c1", "c2", "c3", "c4", "c5"):
            if name == args.workload and not (args.n_workers or args.tensor_list):
                continue
            k = max(3, min(steps, 10 if name in ("c3", "c4", "c5") else 200))
            owl, oms, oout, ows = measure_workload(lib, name, k, 3, flags, 0, 1)
            orows, _, oinfo, _ = kernel_breakdown(lib, owl, k, flags, oout, ows)
            entry = {"workload": name, "n_workers": owl.n_workers, "dtype": owl.spec.dtype,
                     "steps": k, "radices": oinfo["radices"], **summarise(owl, oms, peak),
                     "kernels": [{kk: r[kk] for kk in ("kernel", "level", "radix", "mean_ms", "gbs")} for r in orows]}
            others.append(entry)
            del owl, oout, ows
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": spec.dtype, "data": "synthetic",
            "config": {"workload": args.workload, "n_workers": n_workers, "tensor_list": spec.tensor_list,
                       "num_tensors": num_tensors, "elements_per_worker": total_elems,
                       "radices": info["radices"], "l2": "flushed between steps (512 MB overwritten outside the per-step events)" +
                       ("; inputs also larger than L2" if n_workers * total_elems *
                        workloads.DTYPE_BYTES[spec.dtype] > 2 * 126e6 else ""),
                       "timing": "mean of K per-step CUDA-event intervals on the launching stream",
                       "multi_gpu": "independent replicas of the workload, one per GPU, no collective"},
            "clocks": sampler.summary(), "e2e": e2e, "gpu_launches": steps * info["launches"],
            "roofline": roofline, "cpu_baseline": cpu_baseline,
            "whole_reduce": summary, "variants": variants, "other_workloads": others,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(workloads.SPECS))
    ap.add_argument("--n-workers", type=int, default=0, help="override the configuration's worker count")
    ap.add_argument("--tensor-list", default="", choices=["", "single", "resnet50", "bert_large"],
                    help="override the configuration's tensor list")
    ap.add_argument("--radix-first", type=int, default=0)
    ap.add_argument("--radix-later", type=int, default=0)
    ap.add_argument("--no-level-fusion", action="store_true",
                    help="pass 2 of a level and pass 1 of the next always as separate kernels")
    ap.add_argument("--no-tcgen05", action="store_true", help="radix-64 Gram matrices with mma.sync")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
    else:
        cuda_arm(args)


if __name__ == "__main__":
    main()
