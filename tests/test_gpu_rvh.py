"""Recursive vector-halving Adasum (Algorithm 1) with the GPU arithmetic, all ranks emulated on ONE
GPU in lock step (see rvh_lockstep.py), against the oracle's bottom-up tree with one worker per
rank; and the torch.distributed driver on a one-rank NCCL group."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads
from rvh_lockstep import run_lockstep

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _gradients(size, total, dtype, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [(0.6 * shared + 0.8 * torch.randn(total, generator=gen, device="cuda")).to(TORCH_DT[dtype])
            for _ in range(size)]


@pytest.mark.parametrize("dtype,size,tol", [("f32", 2, 1e-5), ("f32", 4, 1e-5), ("f32", 8, 1e-5), ("f32", 16, 1e-5),
                                            ("f16", 8, 2e-3), ("bf16", 4, 2e-3)])
def test_emulated_ranks_match_the_oracle(dtype, size, tol):
    from paper_2006_02924_b200.rvh import CudaKernels

    offsets = workloads.offsets_from_sizes([300_000, 40, 0, 70_011, 64, 5, 150_000])
    total = int(offsets[-1])
    xs = _gradients(size, total, dtype, seed=2100 + size)
    xs[size - 1][int(offsets[3]):int(offsets[4])] = 0           # one worker's tensor is exactly zero
    kernels = [CudaKernels() for _ in range(size)]
    for k in kernels:
        k.begin()
    results, _ = run_lockstep(size, xs, offsets, kernels)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([_np(x, dtype) for x in xs], offsets=offsets, dtype=dtype, threads=0)
    for r in range(size):
        got = results[r].double().cpu().numpy()
        assert np.all(np.isfinite(got))
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            if hi == lo:
                continue
            err = np.linalg.norm(got[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi])
            assert err <= tol, (r, t, err)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= tol
    # every rank ends with the same bits: the all-gather phase only copies
    assert all(torch.equal(results[0], results[r]) for r in range(1, size))


def test_matches_the_single_gpu_reduce():
    """One worker per rank over 8 emulated ranks = adasum_reduce of the 8 gradients with the
    literal tree (radix 2 at every level), up to fp32 rounding."""
    from paper_2006_02924_b200 import binding as lib
    from paper_2006_02924_b200.rvh import CudaKernels

    offsets = workloads.offsets_from_sizes([200_000, 999, 50_000])
    xs = _gradients(8, int(offsets[-1]), "f32", seed=2200)
    kernels = [CudaKernels() for _ in range(8)]
    for k in kernels:
        k.begin()
    results, _ = run_lockstep(8, xs, offsets, kernels)
    want = lib.adasum_reduce(xs, offsets, flags=lib.flags_radix(2, 2))
    torch.cuda.synchronize()
    assert float(torch.linalg.norm(results[3] - want) / torch.linalg.norm(want)) < 1e-6


def test_driver_with_one_rank_group():
    import torch.distributed as dist
    from paper_2006_02924_b200.rvh import AdasumRVH

    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29672", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
        created = True
    try:
        x = _gradients(1, 10_000, "f16", seed=2300)[0]
        y = AdasumRVH()(x, [0, 4000, 10_000])
        torch.cuda.synchronize()
        assert y.dtype == torch.float32 and torch.equal(y, x.float())
    finally:
        if created:
            dist.destroy_process_group()
