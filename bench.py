#!/usr/bin/env python
"""Benchmark of the N-way Adasum combine.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]

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
    "fingerprint": "0ce4e186d10fa528",
    # "<workload>/<kernel>/<level>": DRAM bytes of the captured launch and the algorithmic bytes of that
    # same launch (captures of the larger configurations are taken on a smaller case of the same kernel
    # and scaled by algorithmic bytes)
    "captures": {
        "c4/gram_partial/0": {"dram_bytes": 3296996376, "algorithmic_bytes": 3271300096,
            "profile": "profiles/gram_partial_tc64_f16_r64_c4_resnet50.txt"},
        "c4:resnet50:n64/gram_partial/0": {"dram_bytes": 3296996376, "algorithmic_bytes": 3271300096,
            "profile": "profiles/gram_partial_tc64_f16_r64_c4_resnet50.txt"},
        "c4/weighted_sum/0": {"dram_bytes": 3333508120, "algorithmic_bytes": 3373528224,
            "profile": "profiles/weighted_sum_f16_r64_c4_resnet50.txt"},
        "c4:resnet50:n64/weighted_sum/0": {"dram_bytes": 3333508120, "algorithmic_bytes": 3373528224,
            "profile": "profiles/weighted_sum_f16_r64_c4_resnet50.txt"},
        "c3/gram_partial/0": {"dram_bytes": 1640642856, "algorithmic_bytes": 1635650048,
            "profile": "profiles/gram_partial_mma_f32_r16_c2_n16.txt"},
        "c5/gram_partial/0": {"dram_bytes": 1640642856, "algorithmic_bytes": 1635650048,
            "profile": "profiles/gram_partial_mma_f32_r16_c2_n16.txt"},
        "c5/gram_partial/1": {"dram_bytes": 1640642856, "algorithmic_bytes": 1635650048,
            "profile": "profiles/gram_partial_mma_f32_r16_c2_n16.txt"},
        "c2:resnet50:n16/gram_partial/0": {"dram_bytes": 1640642856, "algorithmic_bytes": 1635650048,
            "profile": "profiles/gram_partial_mma_f32_r16_c2_n16.txt"},
        "c3/weighted_sum/0": {"dram_bytes": 1692817312, "algorithmic_bytes": 1737878176,
            "profile": "profiles/weighted_sum_f32_r16_c2_n16.txt"},
        "c5/weighted_sum/0": {"dram_bytes": 1692817312, "algorithmic_bytes": 1737878176,
            "profile": "profiles/weighted_sum_f32_r16_c2_n16.txt"},
        "c5/weighted_sum/1": {"dram_bytes": 1692817312, "algorithmic_bytes": 1737878176,
            "profile": "profiles/weighted_sum_f32_r16_c2_n16.txt"},
        "c2:resnet50:n16/weighted_sum/0": {"dram_bytes": 1692817312, "algorithmic_bytes": 1737878176,
            "profile": "profiles/weighted_sum_f32_r16_c2_n16.txt"},
        "c2/gram_partial/0": {"dram_bytes": 821763840, "algorithmic_bytes": 817825024,
            "profile": "profiles/gram_partial_mma_f32_r8_c2.txt"},
        "c2/weighted_sum/0": {"dram_bytes": 871814400, "algorithmic_bytes": 920053152,
            "profile": "profiles/weighted_sum_f32_r8_c2.txt"},
        "c1/fused_small/0": {"dram_bytes": 8084224, "algorithmic_bytes": 12000000,
            "profile": "profiles/fused_small_f32_r2_c1.txt"},
    },
}


def kernel_source_fingerprint() -> str:
    import hashlib

    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2006_02924_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh", ".h")):
            with open(os.path.join(csrc, name), "rb") as fh:
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
    level = plan_levels[record["level"]] if record["level"] < len(plan_levels) else None
    if record["kernel"] == "short_tensors" or level is None:
        return 0                                # a few hundred elements per worker
    elem_bytes = in_bytes if record["level"] == 0 else 4
    read = level["operands"] * total_elems * elem_bytes
    if record["kernel"] == "gram_partial":
        return read
    if record["kernel"] == "weighted_sum":
        return read + level["groups"] * total_elems * 4
    if record["kernel"] in ("fused_small", "fused_l2"):   # both passes in one launch: HBM sees the operands once
        return read + level["groups"] * total_elems * 4
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


class Reducer:
    """One workload on this rank with its output and workspace, and the call that reduces it:
    adasum_reduce, or (several GPUs, every rank holding a slice of every tensor) the element-sharded
    reduce whose Gram sums are all-reduced over NCCL between the two passes of every level."""

    def __init__(self, lib, wl, flags, sharded_group=None, sharded=False):
        self.lib, self.wl, self.flags, self.sharded, self.group = lib, wl, flags, sharded, sharded_group
        dev = wl.grads[0].device
        self.out = torch.empty(wl.total_elems, dtype=torch.float32, device=dev)
        need = lib.adasum_workspace_bytes(wl.total_elems, wl.num_tensors, wl.n_workers, wl.spec.dtype, flags)
        self.ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        self.stream = torch.cuda.current_stream()

    def __call__(self, grads=None):
        grads = self.wl.grads if grads is None else grads
        if self.sharded:
            self.lib.adasum_reduce_sharded(grads, self.wl.offsets, group=self.group, out=self.out, workspace=self.ws,
                                           flags=self.flags, stream=self.stream)
        else:
            self.lib.adasum_reduce(grads, self.wl.offsets, out=self.out, workspace=self.ws, flags=self.flags,
                                   stream=self.stream)


def time_steps(call, steps, warmup, world=1, sampler=None, flush=True, device="cuda"):
    """W warm-up steps, then K timed steps bracketed by barrier + synchronize.  Every step is timed
    with its own pair of CUDA events on the launching stream; between steps a buffer four times the
    size of L2 is overwritten (outside the events), so no step finds its inputs cached by the
    previous one.  Returns ms per step (local): the mean of the K event intervals."""
    import torch.distributed as dist

    scrub = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device) if flush else None
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        call()
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
            call()
            stops[i].record(stream)
        if sampler is not None:
            sampler.sample_once()
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    return sum(a.elapsed_time(b) for a, b in zip(starts, stops)) / steps


def time_variants(lib, wl, steps, warmup, flags):
    """The same workload through adasum_reduce_delta (with a start buffer: the optimizer-delta form,
    result written over the start buffer; and with bf16 output) and through adasum_reduce_scaled.
    Per-step events, L2 flushed."""
    dev = wl.grads[0].device
    dt = wl.grads[0].dtype
    need = lib.adasum_workspace_bytes(wl.total_elems, wl.num_tensors, wl.n_workers, wl.spec.dtype, flags)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
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
    if wl.n_workers >= 2:
        # the same buffers read as scale x gradient (dynamic scaling): one scale per worker and tensor
        scales = torch.exp2(torch.randint(-4, 5, (wl.n_workers, wl.num_tensors), generator=gen, device=dev).float())
        out32 = torch.empty(wl.total_elems, dtype=torch.float32, device=dev)
        cases.append(("scaled reduce, one scale per worker and tensor",
                      lambda: lib.adasum_reduce_scaled(wl.grads, scales, wl.offsets, out=out32, workspace=ws,
                                                       flags=flags, stream=stream),
                      2 * wl.n_workers * wl.total_elems * b + 4 * wl.total_elems))
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
        ms = time_steps(call, steps, warmup, device=dev)
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


def kernel_breakdown(lib, reducer, steps):
    """The same K steps again with an event after every launch; per (kernel, level): launches,
    mean ms, total ms.  Returns (rows sorted by total time, instrumented ms per step, plan info,
    plan levels, launches of this library's kernels per step)."""
    wl = reducer.wl
    info, levels = plan_levels_of(lib, wl, reducer.flags)
    capacity = steps * (max(info["launches"], 1) + 4 * len(levels) + 4) + 8
    lib.adasum_profile_enable(capacity)
    torch.cuda.synchronize()
    scrub = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=reducer.out.device)
    for _ in range(steps):
        scrub.zero_()
        reducer()
    torch.cuda.synchronize()
    del scrub
    records = lib.adasum_profile_collect(capacity)
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
    return rows, sum(g["total_ms"] for g in rows) / steps, info, levels, len(records) / steps


def time_e2e(reducer, steps, world=1):
    """Inputs start in pinned host memory every step and the result is read back to the host: per
    step one host-to-device copy per worker buffer (into the buffers the reduce reads), the reduce,
    one device-to-host copy of the result.  Returns (ms per step, H2D bytes, D2H bytes, check)."""
    import torch.distributed as dist

    wl = reducer.wl
    host_in = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True).copy_(g) for g in wl.grads]
    host_out = torch.empty(wl.total_elems, dtype=torch.float32, pin_memory=True)
    stream = torch.cuda.current_stream()

    def step():
        for d, h in zip(wl.grads, host_in):
            d.copy_(h, non_blocking=True)
        reducer()
        host_out.copy_(reducer.out, non_blocking=True)

    step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.perf_counter()
    t0.record(stream)
    for _ in range(steps):
        step()
    t1.record(stream)
    torch.cuda.synchronize()
    wall = (time.perf_counter() - wall0) * 1e3 / steps
    ms = max(t0.elapsed_time(t1) / steps, wall)
    check = float(host_out[:8].abs().sum())
    del host_in
    return ms, wl.input_bytes, wl.total_elems * 4, check


# ---- the CPU oracle arm ------------------------------------------------------------------------------

def oracle_sample(wl_cpu, budget_elem_ops: float, threads: int = 1):
    """A sample of whole tensors (largest first until the budget is used) whose reduction costs
    about budget_elem_ops = 2 (N-1) * elements.  The oracle's threads each take whole tensors, so
    with `threads` > 1 tensors larger than a thread's share of the budget are passed over (as long
    as smaller ones exist): the sample then keeps every core busy."""
    sizes = np.diff(wl_cpu.offsets)
    per_elem = 2.0 * max(wl_cpu.n_workers - 1, 1)
    order = np.argsort(-sizes, kind="stable")
    share = budget_elem_ops / max(threads, 1)
    if threads > 1 and np.any((sizes > 0) & (per_elem * sizes <= share)):
        order = [t for t in order if per_elem * float(sizes[t]) <= share]
    chosen, used = [], 0.0
    for t in order:
        cost = per_elem * float(sizes[t])
        if sizes[t] == 0 or (chosen and used + cost > budget_elem_ops):
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
    from oracle import adasum_oracle as oracle

    cores = oracle.threads_used(0)
    probe = oracle_sample(wl, 4e8, cores)
    dt, nbytes, threads = run_oracle(wl, probe)
    per_elem = 2.0 * max(spec.n_workers - 1, 1)
    probe_ops = per_elem * sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in probe)
    rate = probe_ops / max(dt, 1e-6)
    budget = rate * min(120.0 / (steps + warmup), 20.0)
    full_ops = per_elem * wl.total_elems
    tensors = all_tensors if budget >= full_ops else oracle_sample(wl, budget, cores)
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


def sharded_local_sizes(spec, world: int, rank: int):
    """Tensor sizes of rank `rank`'s slice when every tensor of the configuration is cut into
    `world` element ranges (workloads.element_shards); a tensor may be empty on the last ranks."""
    offsets = workloads.offsets_from_sizes(spec.tensor_sizes())
    local_offsets, _ = workloads.element_shards(offsets, world)[rank]
    return [int(v) for v in np.diff(local_offsets)]


def allreduce_bytes_per_level(num_tensors: int, levels):
    """Bytes of fp64 Gram sums every rank contributes to the all-reduce of each level."""
    return [num_tensors * lv["groups"] * (lv["radix"] * (lv["radix"] + 1) // 2) * 8 for lv in levels]


def whole_reduce_summary(n_workers, total_elems, elem_bytes, ms, peak):
    """Both readings of "fraction of the HBM roofline" for the whole reduce: the one-read formula
    (N P b read + 4 P written, at peak), which a two-phase method cannot reach for tensors that do
    not fit on chip, and the two-read bound (dot products complete before any output)."""
    one_read = n_workers * total_elems * elem_bytes + 4 * total_elems
    two_read = 2 * n_workers * total_elems * elem_bytes + 4 * total_elems
    per_s = 1.0 / (ms * 1e-3) / 1e9
    return {
        "ms_per_reduce": ms,
        "input_gbs": n_workers * total_elems * elem_bytes * per_s,
        "one_read_bytes": one_read, "two_read_bytes": two_read,
        "one_read_roofline_frac_measured_peak": one_read * per_s / peak,
        "one_read_roofline_frac_nominal_8TBs": one_read * per_s / NOMINAL_HBM_GBS,
        "two_read_roofline_frac_measured_peak": two_read * per_s / peak,
        "two_read_roofline_frac_nominal_8TBs": two_read * per_s / NOMINAL_HBM_GBS,
    }


def traffic_of(workload_key: str, row) -> dict:
    """ncu DRAM bytes per launch for this kernel, scaled from the captured case by algorithmic
    bytes (traffic grows in proportion: every operand byte crosses HBM once per pass); None once
    the kernel sources have changed since the counters were taken."""
    if NCU_TRAFFIC["fingerprint"] != kernel_source_fingerprint():
        return None
    entry = NCU_TRAFFIC["captures"].get(f"{workload_key}/{row['kernel']}/{row['level']}")
    if entry is None or entry["algorithmic_bytes"] <= 0:
        return None
    return int(round(entry["dram_bytes"] * row["bytes_per_launch"] / entry["algorithmic_bytes"]))


def cpu_baseline_of(wl, name: str, seconds: float):
    """The fp64 oracle, as it stands, on a bounded sample of the workload (whole tensors), sized from
    a short calibration run so that it takes about `seconds` on this host."""
    from oracle import adasum_oracle as oracle

    threads = oracle.threads_used(0)
    per_elem = 2.0 * max(wl.n_workers - 1, 1)
    full_ops = per_elem * wl.total_elems
    probe = oracle_sample(wl, min(full_ops, 4e8), threads)
    dt, _, _ = run_oracle(wl, probe)
    probe_ops = per_elem * sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in probe)
    budget = probe_ops / max(dt, 1e-6) * seconds
    # at most 16 GB of inputs are staged on the host
    budget = min(budget, per_elem * 16e9 / (wl.n_workers * workloads.DTYPE_BYTES[wl.spec.dtype]))
    cap = per_elem * 16e9 / (wl.n_workers * workloads.DTYPE_BYTES[wl.spec.dtype])
    tensors = list(range(wl.num_tensors)) if budget >= full_ops else oracle_sample(wl, budget, threads)
    dt, nbytes, used = run_oracle(wl, tensors)
    if dt < 0.4 * seconds and len(tensors) < wl.num_tensors and budget < cap:
        # the short calibration run under-estimated the rate (start-up costs): one larger sample
        budget = min(budget * min(seconds / max(dt, 1e-3), 8.0), cap)
        tensors = list(range(wl.num_tensors)) if budget >= full_ops else oracle_sample(wl, budget, threads)
        dt, nbytes, used = run_oracle(wl, tensors)
    elems = sum(int(wl.offsets[t + 1] - wl.offsets[t]) for t in tensors)
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"{len(tensors)} of {wl.num_tensors} tensors of {name}, {elems} elements x "
                      f"{wl.n_workers} workers ({nbytes / 1e9:.2f} GB of inputs), {dt:.2f} s"}


def measure_config(lib, name, spec, steps, warmup, flags, peak, peak_kind, *, world=1, rank=0, mode="single",
                   sampler=None, e2e_steps=3, cpu_seconds=10.0, tensor_sizes=None, traffic_key=None):
    """One configuration end to end: the timed steps, the per-launch breakdown with the roofline of
    the dominant kernel, the end-to-end leg and (one GPU only) the CPU oracle beside it."""
    sharded = mode == "sharded"
    wl = workloads.generate(spec, device="cuda", tensor_sizes=tensor_sizes, replica=rank)
    reducer = Reducer(lib, wl, flags, sharded=sharded)
    ms_local = time_steps(reducer, steps, warmup, world=world, sampler=sampler)
    eb = workloads.DTYPE_BYTES[spec.dtype]
    if sharded:          # strong scaling: the job is the whole configuration, the time the slowest rank's
        job_elems = sum(spec.tensor_sizes())
        ms, _ = aggregate_over_ranks(ms_local, 0.0, world, "cuda")
        job_bytes = float(spec.n_workers * job_elems * eb)
    else:
        job_elems = wl.total_elems * world
        ms, job_bytes = aggregate_over_ranks(ms_local, float(wl.input_bytes), world, "cuda")
    rows, ms_instrumented, info, levels, launches_per_step = kernel_breakdown(lib, reducer, steps)
    top = rows[0]
    total_rows_ms = sum(r["total_ms"] for r in rows)
    roofline = {
        "bound": "hbm", "kernel": f"{top['kernel']}<radix {top['radix']}> level {top['level']}",
        "achieved": top["gbs"], "peak": peak, "unit": "GB/s", "frac": top["gbs"] / peak,
        "peak_kind": f"of {peak_kind}", "traffic": traffic_of(traffic_key or name, top),
        "bytes_per_launch": top["bytes_per_launch"], "mean_launch_ms": top["mean_ms"],
        "share_of_step": top["total_ms"] / total_rows_ms if total_rows_ms > 0 else None,
        "timing": "CUDA event after every launch, same K steps (L2 flushed between them) repeated right "
                  "after the timed region",
        "instrumented_ms_per_step": ms_instrumented,
        "kernels": [dict({k: r[k] for k in ("kernel", "level", "radix", "launches", "mean_ms", "gbs")},
                         frac=r["gbs"] / peak, traffic=traffic_of(traffic_key or name, r)) for r in rows],
        "whole_reduce": whole_reduce_summary(spec.n_workers, job_elems if sharded else wl.total_elems, eb,
                                             ms if sharded else ms_local, peak),
    }
    e2e = None
    if e2e_steps > 0:
        e2e_ms_local, h2d, d2h, _ = time_e2e(reducer, e2e_steps, world=world)
        e2e_ms, _ = aggregate_over_ranks(e2e_ms_local, 0.0, world, "cuda")
        e2e = {"value": job_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "bytes_are": "per rank" if world > 1 else "whole job"}
    cpu_baseline = None
    if rank == 0 and world == 1 and cpu_seconds > 0:
        cpu_baseline = cpu_baseline_of(wl, name, cpu_seconds)
    entry = {
        "workload": name, "n_workers": spec.n_workers, "dtype": spec.dtype, "tensor_list": spec.tensor_list,
        "num_tensors": wl.num_tensors, "elements_per_worker": job_elems if sharded else wl.total_elems,
        "steps": steps, "radices": info["radices"], "ms_per_reduce": ms,
        "input_gbs": job_bytes / (ms * 1e-3) / 1e9, "launches_per_step": launches_per_step,
        "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline,
    }
    if sharded:
        entry["allreduce_bytes_per_level"] = allreduce_bytes_per_level(wl.num_tensors, levels)
    return entry, wl, reducer


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
    elif args.force_multi:          # the multi-GPU code path on a group of one rank
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29687", rank=0, world_size=1,
                                device_id=torch.device("cuda", local_rank))
    from paper_2006_02924_b200 import binding as lib

    flags = lib.flags_radix(args.radix_first, args.radix_later)
    if args.no_level_fusion:
        flags |= lib.ADASUM_FLAG_NO_LEVEL_FUSION
    if args.no_tcgen05:
        flags |= lib.ADASUM_FLAG_NO_TCGEN05
    peak, peak_kind = measured_peak()
    sampler = ClockSampler(local_rank)
    steps, warmup = max(args.steps, 1), max(args.warmup, 3)
    mode = "single" if world == 1 and not args.force_multi else args.multi
    single = rank == 0 and world == 1

    main_spec = resolve_spec(args.workload, args.n_workers, args.tensor_list)
    sizes = sharded_local_sizes(main_spec, world, rank) if mode == "sharded" else None
    overridden = bool(args.n_workers or args.tensor_list)
    traffic_key = args.workload if not overridden else \
        f"{args.workload}:{main_spec.tensor_list}:n{main_spec.n_workers}"
    head, wl, reducer = measure_config(
        lib, args.workload, main_spec, steps, warmup, flags, peak, peak_kind, world=world, rank=rank, mode=mode,
        sampler=sampler, e2e_steps=args.e2e_steps, cpu_seconds=0.0 if args.no_cpu_baseline else args.cpu_seconds,
        tensor_sizes=sizes, traffic_key=traffic_key)
    variants = []
    if single and not args.no_other_workloads:
        del reducer
        variants = time_variants(lib, wl, max(3, min(steps, 50)), 3, flags)
    reducer = None
    del wl
    torch.cuda.empty_cache()

    others = []
    if single and not args.no_other_workloads:
        for name in ("c1", "c2", "c3", "c4", "c5"):
            if name == args.workload and not overridden:
                continue
            k = max(3, min(steps, 20 if name in ("c3", "c4", "c5") else 200))
            entry, owl, ored = measure_config(lib, name, workloads.SPECS[name], k, 3, flags, peak, peak_kind,
                                              e2e_steps=args.e2e_steps,
                                              cpu_seconds=0.0 if args.no_cpu_baseline else min(args.cpu_seconds, 6.0))
            others.append(entry)
            del owl, ored
            torch.cuda.empty_cache()

    if rank == 0:
        spec = main_spec
        scaling = "strong" if mode == "sharded" else "weak"
        multi = {"single": "one GPU",
                 "sharded": "every rank holds one element range of every tensor; per level the fp64 Gram sums are "
                            "all-reduced over NCCL between the two passes (no other exchange)",
                 "replicas": "independent replicas of the workload, one per GPU, no collective"}[mode]
        line = {
            "metric": METRIC, "value": head["input_gbs"], "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": head["ms_per_reduce"], "higher_is_better": True, "scaling": scaling,
            "vs_baseline": None, "dtype": spec.dtype, "data": "synthetic",
            "config": {"workload": args.workload, "n_workers": spec.n_workers, "tensor_list": spec.tensor_list,
                       "num_tensors": head["num_tensors"], "elements_per_worker": head["elements_per_worker"],
                       "radices": head["radices"],
                       "l2": "flushed between steps (512 MB overwritten outside the per-step events); inputs are also "
                             "larger than L2" if spec.n_workers * head["elements_per_worker"] *
                             workloads.DTYPE_BYTES[spec.dtype] > 2 * 126e6 else
                             "flushed between steps (512 MB overwritten outside the per-step events)",
                       "timing": "mean of K per-step CUDA-event intervals on the launching stream, max over ranks",
                       "multi_gpu": multi},
            "clocks": sampler.summary(), "e2e": head["e2e"],
            "gpu_launches": int(round(steps * head["launches_per_step"])),
            "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"],
            "variants": variants, "other_workloads": others,
        }
        if "allreduce_bytes_per_level" in head:
            line["config"]["allreduce_bytes_per_level"] = head["allreduce_bytes_per_level"]
        print(json.dumps(line))
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(workloads.SPECS))
    ap.add_argument("--multi", default="sharded", choices=["sharded", "replicas"],
                    help="with several GPUs: every rank holds a slice of every tensor and the Gram sums are "
                         "all-reduced (sharded), or every rank reduces an independent copy of the workload (replicas)")
    ap.add_argument("--force-multi", action="store_true",
                    help="with one GPU: run the --multi code path all the same, on a process group of one rank")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=12.0,
                    help="about how long the CPU oracle runs on its sample of the headline workload")
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
