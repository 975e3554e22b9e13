"""GPU parity of the kernel that does the second pass of one level and the first pass of the next
(Algorithm 1's "apply" of a level and the dot products of the level above it) against the fp64
oracle and against the same plan run as separate kernels."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu

TORCH_DT = workloads.TORCH_DTYPES
NO_FUSION = 1 << 21
TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
# several segments and a ragged tail, tensors shorter than a vector, an empty one, odd starts
SIZES = [70_001, 0, 33, 4099, 1024, 7, 20_000, 2048, 513]


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _correlated(n, total, dtype, seed, rho=0.4):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [((rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device="cuda"))
            .to(TORCH_DT[dtype]) for _ in range(n)]


def _check(out, grads, offsets, dtype, tol):
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0)
    got = out.float().cpu().numpy().astype(np.float64)
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        norm = np.linalg.norm(ref[lo:hi])
        if norm == 0.0:
            assert not got[lo:hi].any(), t
        else:
            err = np.linalg.norm(got[lo:hi] - ref[lo:hi]) / norm
            assert err <= tol, (t, hi - lo, err)


def _kernels(lib, fn):
    lib.adasum_profile_enable(256)
    out = fn()
    torch.cuda.synchronize()
    # the tensors of at most 64 elements have a kernel of their own, launched last; it is not what these tests count
    return out, [r["kernel"] for r in lib.adasum_profile_collect(256) if r["kernel"] != "short_tensors"]


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n,radices", [(2, (2, 2)), (4, (2, 2)), (8, (2, 2)), (3, (2, 2)), (5, (2, 2)), (7, (2, 2)),
                                       (16, (4, 4)), (13, (4, 2)), (12, (2, 4)), (64, (4, 4)), (100, (4, 2)),
                                       (37, (2, 2)), (256, (16, 4))])
def test_level_fusion_parity(lib, dtype, n, radices):
    offsets = workloads.offsets_from_sizes(SIZES)
    grads = _correlated(n, int(offsets[-1]), dtype, seed=4100 + n)
    for g in grads[: n // 2]:
        g[int(offsets[6]):int(offsets[7])] = 0                 # a tensor that is zero on half the workers
    for g in grads:
        g[int(offsets[3]):int(offsets[4])] = 0                 # and one that is zero everywhere
    flags = lib.flags_radix(*radices)
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets, flags=flags))
    levels = lib.adasum_plan_info(int(offsets[-1]), len(SIZES), n, grads[0].dtype, flags)["radices"]
    if len(levels) > 1 and radices[0] <= 4:
        assert "wsum_gram" in kernels, kernels
        assert kernels.count("gram_partial") == 1, kernels       # only the first level runs a pass 1 of its own
    elif len(levels) > 1:                                        # a wide first level keeps its own second pass
        assert kernels[:2] == ["gram_partial", "weighted_sum"] and "wsum_gram" in kernels[2:], kernels
    _check(out, grads, offsets, dtype, TOL[dtype])
    apart, kernels_apart = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets, flags=flags | NO_FUSION))
    assert "wsum_gram" not in kernels_apart
    norm = float(apart.double().norm())
    assert float((out.double() - apart.double()).norm()) <= 10 * TOL[dtype] * norm
    again = lib.adasum_reduce(grads, offsets, flags=flags)
    assert torch.equal(out, again)                                 # deterministic


def test_level_fusion_launch_count_matches_plan(lib):
    offsets = workloads.offsets_from_sizes(SIZES)
    total = int(offsets[-1])
    for n, radices in ((8, (2, 2)), (64, (16, 4)), (300, (2, 2)), (300, (4, 4))):
        grads = _correlated(n, total, "f32", seed=4200 + n, rho=0.1)
        flags = lib.flags_radix(*radices)
        out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets, flags=flags))
        info = lib.adasum_plan_info(total, len(SIZES), n, torch.float32, flags)
        assert len(kernels) == info["launches"], (n, radices, kernels, info)
        _check(out, grads, offsets, "f32", 1e-5)


def test_level_fusion_orthogonality(lib):
    offsets = workloads.offsets_from_sizes([30_000, 33, 4099])
    grads = _correlated(16, int(offsets[-1]), "f32", seed=4300)
    (out, ortho), kernels = _kernels(lib, lambda: lib.adasum_reduce_ex(grads, offsets, flags=lib.flags_radix(2, 2)))
    assert "wsum_gram" in kernels
    _, ref_ortho = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32",
                                        return_orthogonality=True, threads=0)
    assert np.allclose(ortho.cpu().numpy(), ref_ortho, rtol=1e-4)


def test_level_fusion_unaligned_buffers_run_unfused(lib):
    total = 50_001
    base = [torch.randn(total + 1, device="cuda") for _ in range(8)]
    grads = [b[1:] for b in base]
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, flags=lib.flags_radix(2, 2)))
    assert "wsum_gram" not in kernels
    _check(out, grads, np.array([0, total], dtype=np.int64), "f32", 1e-5)


def test_level_fusion_delta_form(lib):
    """The first level of the delta form keeps its own pass 2 (it reads operand - start); later levels fuse."""
    offsets = workloads.offsets_from_sizes([30_000, 33, 4099])
    total = int(offsets[-1])
    start = torch.randn(total, device="cuda")
    currents = [start + 0.01 * g for g in _correlated(8, total, "f32", seed=4400)]
    flags = lib.flags_radix(2, 2)
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce_delta(currents, start, offsets, flags=flags))
    assert kernels.count("wsum_gram") == 1, kernels
    ref = oracle.adasum_reduce_delta([_np(c, "f32") for c in currents], _np(start, "f32"), offsets=offsets,
                                     dtype="f32", threads=0)
    r = ref - _np(start, "f32").astype(np.float64)
    err = np.linalg.norm(out.cpu().numpy().astype(np.float64) - ref)
    assert err <= 1e-5 * np.linalg.norm(r) + 2.0 ** -24 * np.linalg.norm(ref)
