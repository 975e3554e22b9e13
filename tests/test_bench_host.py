"""Host-side logic of bench.py that runs without a GPU: the multi-rank aggregation (gloo, two
ranks), the oracle sampling, the roofline byte counts and the reference arm's rank handling."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2006_02924_b200 import workloads  # noqa: E402


def _rank_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, total = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), world, "cpu")
    results[rank] = (ms, total)
    dist.barrier()
    dist.destroy_process_group()


def test_aggregation_takes_slowest_rank_and_sums_work():
    world = 2
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_rank_main, args=(world, 29653, results), nprocs=world, join=True)
        assert results[0] == results[1] == (15.0, 3000.0)
    assert bench.aggregate_over_ranks(7.0, 11.0, 1) == (7.0, 11.0)


def test_algorithmic_bytes_per_launch():
    levels = [{"radix": 16, "operands": 256, "groups": 16}, {"radix": 16, "operands": 16, "groups": 1}]
    p = 1000
    assert bench.algorithmic_bytes({"kernel": "gram_partial", "level": 0}, levels, p, 2) == 256 * p * 2
    assert bench.algorithmic_bytes({"kernel": "weighted_sum", "level": 0}, levels, p, 2) == 256 * p * 2 + 16 * p * 4
    assert bench.algorithmic_bytes({"kernel": "gram_partial", "level": 1}, levels, p, 2) == 16 * p * 4
    assert bench.algorithmic_bytes({"kernel": "weighted_sum", "level": 1}, levels, p, 2) == 16 * p * 4 + p * 4
    assert bench.algorithmic_bytes({"kernel": "tree_weights", "level": 0}, levels, p, 2) == 0
    one = [{"radix": 2, "operands": 2, "groups": 1}]
    assert bench.algorithmic_bytes({"kernel": "fused_small", "level": 0}, one, p, 4) == 2 * p * 4 + p * 4


def test_oracle_sample_is_bounded_and_whole_tensors():
    wl = workloads.generate("c2", tensor_sizes=workloads.reduced_sizes(workloads.resnet50_tensor_sizes(), 64))
    budget = 2.0 * 7 * 50_000
    chosen = bench.oracle_sample(wl, budget)
    sizes = np.diff(wl.offsets)
    assert chosen == sorted(set(chosen)) and len(chosen) >= 1
    assert 2.0 * 7 * sizes[chosen].sum() <= budget + 2.0 * 7 * sizes.max()
    dt, nbytes, threads = bench.run_oracle(wl, chosen, threads=1)
    assert nbytes == 8 * int(sizes[chosen].sum()) * 4 and dt > 0 and threads == 1


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_element_shards_cover_every_tensor_once():
    offsets = workloads.offsets_from_sizes([1000, 3, 0, 130, 64])
    for world in (1, 2, 3, 8):
        shards = workloads.element_shards(offsets, world)
        assert len(shards) == world
        for t in range(len(offsets) - 1):
            cursor = int(offsets[t])
            for local_offsets, pieces in shards:
                lo, hi = pieces[t]
                assert lo == cursor and hi >= lo
                assert int(local_offsets[t + 1] - local_offsets[t]) == hi - lo
                cursor = hi
            assert cursor == int(offsets[t + 1])


def _sharded_rank_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = workloads.SPECS["c2"]
    local = torch.tensor(bench.sharded_local_sizes(spec, world, rank), dtype=torch.int64)
    summed = local.clone()
    dist.all_reduce(summed, op=dist.ReduceOp.SUM)             # the ranks' slices add up to every tensor
    # strong scaling: the job is the whole configuration, the step time the slowest rank's
    ms, _ = bench.aggregate_over_ranks(3.0 + rank, 0.0, world, "cpu")
    results[rank] = (summed.tolist(), int(local.sum()), ms)
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_mode_slices_and_aggregates_over_two_ranks():
    world = 2
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_sharded_rank_main, args=(world, 29655, results), nprocs=world, join=True)
        sizes = workloads.SPECS["c2"].tensor_sizes()
        assert results[0][0] == results[1][0] == sizes
        assert results[0][1] + results[1][1] == sum(sizes)
        assert results[0][1] >= results[1][1] > 0.4 * sum(sizes)      # balanced up to the 64-element grid
        assert results[0][2] == results[1][2] == 4.0


def test_allreduce_bytes_per_level():
    levels = [{"radix": 16, "operands": 256, "groups": 16}, {"radix": 16, "operands": 16, "groups": 1}]
    assert bench.allreduce_bytes_per_level(161, levels) == [161 * 16 * 136 * 8, 161 * 136 * 8]


def test_whole_reduce_summary_gives_both_readings():
    s = bench.whole_reduce_summary(64, 1000, 2, 1.0, 6000.0)
    assert s["one_read_bytes"] == 64 * 1000 * 2 + 4000 and s["two_read_bytes"] == 2 * 64 * 1000 * 2 + 4000
    assert abs(s["one_read_roofline_frac_measured_peak"] - s["one_read_bytes"] / 1e-3 / 1e9 / 6000.0) < 1e-12
    assert s["two_read_roofline_frac_measured_peak"] > s["one_read_roofline_frac_measured_peak"]
