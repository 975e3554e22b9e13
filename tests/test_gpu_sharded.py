"""The element-sharded reduce (every GPU holds a slice of every tensor, one all-reduce of the Gram
sums per level), checked on ONE GPU: the ranks' calls are made one after the other and the
all-reduce is a plain sum of their Gram sums.  No kernel waits for another one, so this is exactly
what G processes would compute."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _inputs(n, total, dtype, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [(0.7 * shared + 0.7 * torch.randn(total, generator=gen, device="cuda")).to(TORCH_DT[dtype])
            for _ in range(n)]


@pytest.mark.parametrize("dtype,n,world,flags,tol", [
    ("f32", 8, 2, 0, 1e-5), ("f32", 20, 3, 0, 1e-5), ("f16", 64, 4, 0, 2e-3), ("bf16", 40, 2, 0, 2e-3),
    ("f32", 64, 3, 16 | (4 << 8), 1e-5), ("f32", 12, 2, 1 << 18, 1e-5)])
def test_emulated_ranks_match_the_oracle(lib, dtype, n, world, flags, tol):
    offsets = workloads.offsets_from_sizes([100_000, 40, 0, 30_011, 64, 5])
    total = int(offsets[-1])
    grads = _inputs(n, total, dtype, seed=1200 + n)
    shards = workloads.element_shards(offsets, world)
    ranks = []
    for local_offsets, pieces in shards:
        local = [torch.cat([g[lo:hi] for lo, hi in pieces]).contiguous() for g in grads]
        need = lib.adasum_workspace_bytes(int(local_offsets[-1]), len(pieces), n, dtype, flags)
        ranks.append({
            "offsets": local_offsets, "pieces": pieces, "grads": local,
            "ws": torch.empty(max(need, 256), dtype=torch.uint8, device="cuda"),
            "out": torch.full((max(int(local_offsets[-1]), 1),), float("nan"), device="cuda")[:int(local_offsets[-1])],
            "ortho": torch.empty(len(pieces), device="cuda"),
        })
    assert any(hi == lo for r in ranks[1:] for lo, hi in r["pieces"][1:2])      # the 40-element tensor is on rank 0 only
    levels = len(lib.adasum_plan_info(total, len(offsets) - 1, n, dtype, flags)["radices"])
    for level in range(levels):
        sums = [lib.adasum_sharded_gram(r["grads"], r["offsets"], r["ws"], level, flags=flags) for r in ranks]
        total_sums = torch.stack([s.clone() for s in sums]).sum(dim=0)       # the all-reduce
        for s in sums:
            s.copy_(total_sums)
        for r in ranks:
            lib.adasum_sharded_apply(r["grads"], r["offsets"], r["out"], r["ws"], level,
                                     orthogonality=r["ortho"], flags=flags)
    torch.cuda.synchronize()
    got = np.full(total, np.nan)
    for r in ranks:
        o = r["out"].cpu().numpy()
        for t, (lo, hi) in enumerate(r["pieces"]):
            a = int(r["offsets"][t])
            got[lo:hi] = o[a:a + hi - lo]
    ref, ref_ortho = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype,
                                          linear_order=bool(flags & (1 << 18)), return_orthogonality=True,
                                          threads=0)
    assert np.all(np.isfinite(got))
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        err = np.linalg.norm(got[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi])
        assert err <= tol, (t, err)
        for r in ranks:         # every rank derives the same measure from the summed matrices
            assert abs(float(r["ortho"][t]) - ref_ortho[t]) <= max(10 * tol, 1e-4) * ref_ortho[t]
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= tol


def test_single_process_group_driver(lib):
    """adasum_reduce_sharded with a one-rank process group equals adasum_reduce."""
    import torch.distributed as dist

    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29671", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
        created = True
    try:
        offsets = workloads.offsets_from_sizes([60_000, 33, 9000])
        grads = _inputs(24, int(offsets[-1]), "f32", seed=1300)
        got = lib.adasum_reduce_sharded(grads, offsets)
        want = lib.adasum_reduce(grads, offsets)
        torch.cuda.synchronize()
        assert float(torch.linalg.norm(got - want) / torch.linalg.norm(want)) < 1e-6
    finally:
        if created:
            dist.destroy_process_group()


def test_level_outside_the_plan_is_refused(lib):
    grads = _inputs(4, 1000, "f32", seed=1400)
    ws = torch.empty(lib.adasum_workspace_bytes(1000, 1, 4, "f32"), dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.AdasumError):
        lib.adasum_sharded_gram(grads, [0, 1000], ws, 1)
