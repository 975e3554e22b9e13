"""Recursive vector-halving across ranks (Algorithm 1): the schedule, the per-rank step sequence
and the torch.distributed driver, on the CPU.  The arithmetic is replaced by a small fp64 stand-in
defined here, because the product's arithmetic exists on the GPU only; what these tests pin is
who exchanges which element range with whom, which ranks add their partial sums, and that the
whole procedure reproduces the bottom-up tree of the oracle with one worker per rank."""
import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads
from paper_2006_02924_b200.rvh import AdasumRVH, clip_offsets, rvh_schedule
from rvh_lockstep import run_lockstep


class DoubleKernels:
    """fp64 stand-in for the GPU arithmetic (test double)."""

    def empty(self, n, dtype, like):
        return torch.empty(int(n), dtype=dtype)

    def result(self, n, like):
        return torch.empty(int(n), dtype=torch.float32)

    def gram(self, a, b, offsets, level):
        a, b = a.double(), b.double()
        sums = torch.zeros(3 * (len(offsets) - 1), dtype=torch.float64)
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            sums[3 * t] = (a[lo:hi] * a[lo:hi]).sum()
            sums[3 * t + 1] = (a[lo:hi] * b[lo:hi]).sum()
            sums[3 * t + 2] = (b[lo:hi] * b[lo:hi]).sum()
        self.sums = sums
        return sums

    def apply(self, a, b, offsets, level):
        out = torch.empty(a.numel(), dtype=torch.float64)
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            aa, ab, bb = (float(v) for v in self.sums[3 * t:3 * t + 3])
            ca = 1.0 if aa == 0.0 else 1.0 - ab / (2.0 * aa)
            cb = 1.0 if bb == 0.0 else 1.0 - ab / (2.0 * bb)
            out[lo:hi] = ca * a[lo:hi].double() + cb * b[lo:hi].double()
        return out


@pytest.mark.parametrize("size", [1, 2, 4, 8, 32])
@pytest.mark.parametrize("total", [33, 1000, 4096 + 17, 1_000_003])
def test_schedule_is_consistent(size, total):
    if total < size:
        pytest.skip("fewer elements than ranks")
    sched = [rvh_schedule(r, size, total) for r in range(size)]
    levels = size.bit_length() - 1
    assert all(len(s) == levels for s in sched)
    for r in range(size):
        for lv in sched[r]:
            peer = sched[lv.neighbor][sched[r].index(lv)]
            assert peer.neighbor == r and peer.left != lv.left
            assert (peer.lo, peer.mid, peer.hi) == (lv.lo, lv.mid, lv.hi)      # both hold the same range
            assert peer.give == lv.keep and peer.keep == lv.give
            assert lv.lo < lv.mid < lv.hi
            assert len(lv.group) == 2 * lv.distance and r in lv.group and lv.neighbor in lv.group
            assert lv.group[0] % (2 * lv.distance) == 0
            # the group's ranks together hold the whole vector exactly once after this level
            held = sorted(sched[q][sched[r].index(lv)].keep for q in lv.group)
            if lv.distance == 1:
                assert held == [(lv.lo, lv.mid), (lv.mid, lv.hi)]
    # after the last level the ranks' ranges partition [0, total)
    if levels:
        final = sorted(s[-1].keep for s in sched)
        assert final[0][0] == 0 and final[-1][1] == total
        assert all(final[i][1] == final[i + 1][0] for i in range(size - 1))


def test_schedule_refuses_what_algorithm_1_excludes():
    with pytest.raises(ValueError):
        rvh_schedule(0, 6, 1000)
    with pytest.raises(ValueError):
        rvh_schedule(4, 4, 1000)
    with pytest.raises(ValueError):
        rvh_schedule(0, 8, 7)


def test_clip_offsets():
    offs = [0, 10, 10, 25, 40]
    assert clip_offsets(offs, 0, 40).tolist() == offs
    assert clip_offsets(offs, 12, 30).tolist() == [0, 0, 0, 13, 18]
    assert clip_offsets(offs, 25, 40).tolist() == [0, 0, 0, 0, 15]


def _gradients(size, total, seed):
    rng = np.random.default_rng(seed)
    shared = rng.standard_normal(total)
    return [(0.6 * shared + 0.8 * rng.standard_normal(total)).astype(np.float32) for _ in range(size)]


@pytest.mark.parametrize("size", [1, 2, 4, 8, 16])
def test_lockstep_equals_the_tree_of_the_oracle(size):
    offsets = workloads.offsets_from_sizes([700, 3, 0, 1290, 64, 5000, 1])
    total = int(offsets[-1])
    xs = _gradients(size, total, seed=size)
    xs[size // 2][int(offsets[3]):int(offsets[4])] = 0.0            # a zero operand inside the tree
    results, log = run_lockstep(size, [torch.from_numpy(x) for x in xs], offsets,
                                [DoubleKernels() for _ in range(size)])
    ref = oracle.adasum_reduce(xs, offsets=offsets, dtype="f32", threads=1)
    for r in range(size):
        got = results[r].double().numpy()
        assert np.linalg.norm(got - ref) <= 2e-7 * np.linalg.norm(ref), r
    levels = size.bit_length() - 1
    assert [k[0] for k in log] == ["exchange", "allreduce"] * levels + ["exchange"] * levels
    # halving: each exchange of the first phase moves half of what the previous one did
    sent = [k[2][0] for k in log if k[0] == "exchange"][:levels]
    assert all(abs(sent[i] - total / 2 ** (i + 1)) <= 64 for i in range(levels))


def _rank_main(rank, world, port, offsets, xs, out):
    import torch.distributed as dist

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        reduce = AdasumRVH(kernels=DoubleKernels())
        y = reduce(torch.from_numpy(xs[rank]), offsets)
        y2 = reduce(torch.from_numpy(xs[rank]), offsets)         # a second reduce reuses the sub-groups
        assert torch.equal(y, y2)
        out[rank] = y.numpy()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_driver_over_gloo(world):
    offsets = workloads.offsets_from_sizes([3000, 17, 0, 2048])
    total = int(offsets[-1])
    xs = _gradients(world, total, seed=40 + world)
    with mp.Manager() as manager:
        out = manager.dict()
        mp.spawn(_rank_main, args=(world, 29700 + world, offsets, xs, out), nprocs=world, join=True)
        ref = oracle.adasum_reduce(xs, offsets=offsets, dtype="f32", threads=1)
        for r in range(world):
            assert np.linalg.norm(out[r].astype(np.float64) - ref) <= 2e-7 * np.linalg.norm(ref)
        assert all(np.array_equal(out[0], out[r]) for r in range(world))


def test_gpu_arithmetic_refuses_cpu_tensors():
    from paper_2006_02924_b200.rvh import CudaKernels

    try:
        kernels = CudaKernels()
    except ImportError:
        pytest.skip("native library not built")
    with pytest.raises(RuntimeError):
        kernels.empty(8, torch.float32, torch.zeros(8))
