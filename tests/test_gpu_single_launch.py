"""The single cooperative launch that serves one-level reduces of at most 8 workers whose operands fit
the L2: long tensors are cut into one segment per block (operands kept in registers across the grid
barrier when the segment is short enough), tensors of 65 to 512 elements are reduced by one warp
each, and those of at most 64 elements by the fp64 kernel.  Against the fp64 oracle at the plain
tolerance, every tensor."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES
TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
LINEAR, TOP_DOWN = 1 << 18, 1 << 20


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _correlated(n, total, dtype, seed, rho=0.3):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [((rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device="cuda"))
            .to(TORCH_DT[dtype]) for _ in range(n)]


def _kernels(lib, fn):
    lib.adasum_profile_enable(64)
    out = fn()
    torch.cuda.synchronize()
    return out, [r["kernel"] for r in lib.adasum_profile_collect(64)]


def _check(out, ref, offsets, tol):
    out = out.double().cpu().numpy()
    assert np.all(np.isfinite(out))
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        nr = np.linalg.norm(ref[lo:hi])
        if nr == 0.0:
            assert not out[lo:hi].any(), t
            continue
        err = np.linalg.norm(out[lo:hi] - ref[lo:hi]) / nr
        assert err <= tol, f"tensor {t} (len {hi - lo}): rel-L2 {err:.3e} > {tol:.1e}"


# long, warp-sized and short tensors, ragged lengths, an empty one
MIXED = [300_000, 2048, 2049, 65, 64, 0, 1000, 7, 129, 40_001, 1, 2047, 513]


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", [2, 3, 4, 5, 8])
def test_mixed_tensor_sizes(lib, dtype, n):
    offsets = workloads.offsets_from_sizes(MIXED)
    grads = _correlated(n, int(offsets[-1]), dtype, seed=7000 + n)
    for g in grads[: n // 2]:
        g[int(offsets[6]):int(offsets[7])] = 0                # a warp-sized tensor that is zero on some workers
    for g in grads:
        g[int(offsets[12]):int(offsets[13])] = 0              # and one that is zero everywhere
    (out, ortho), kernels = _kernels(lib, lambda: lib.adasum_reduce_ex(grads, offsets))
    assert kernels == ["fused_small"], kernels       # the short tensors included
    ref, ref_ortho = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0,
                                          return_orthogonality=True)
    _check(out, ref, offsets, TOL[dtype])
    got = ortho.double().cpu().numpy()
    for t, size in enumerate(MIXED):
        if size == 0 or t == 12:
            assert np.isnan(got[t]), t
        else:
            assert abs(got[t] - ref_ortho[t]) <= max(10 * TOL[dtype], 1e-4) * ref_ortho[t], (t, got[t], ref_ortho[t])
    assert torch.equal(out, lib.adasum_reduce(grads, offsets))          # deterministic


@pytest.mark.parametrize("dtype,n", [("f32", 2), ("f32", 4), ("f16", 8), ("bf16", 4)])
def test_a_fused_buffer_of_many_tensors(lib, dtype, n):
    """The 161 tensors of ResNet-50 at an eighth of their size (3.2 M elements, 107 of them small):
    one launch, not one block per tensor."""
    sizes = workloads.reduced_sizes(workloads.resnet50_tensor_sizes(), 8)
    wl = workloads.generate("c2", device="cuda", tensor_sizes=sizes, n_workers=n)
    grads = [g.to(TORCH_DT[dtype]) for g in wl.grads]
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, wl.offsets))
    assert kernels == ["fused_small"], kernels
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=wl.offsets, dtype=dtype, threads=0)
    _check(out, ref, wl.offsets, TOL[dtype])


def test_only_small_tensors(lib):
    sizes = [100, 2048, 65, 999, 64, 3]
    offsets = workloads.offsets_from_sizes(sizes)
    grads = _correlated(4, int(offsets[-1]), "f32", seed=7100)
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets))
    assert kernels == ["fused_small"], kernels       # the short tensors included
    ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32", threads=0)
    _check(out, ref, offsets, 1e-5)


@pytest.mark.parametrize("n,total", [(2, 1_000_000), (2, 4_000_000), (4, 3_000_001), (8, 2_500_000), (2, 11_000_000)])
def test_one_long_tensor(lib, n, total):
    """Segments short enough to stay in registers, and longer ones that are read again out of the L2."""
    grads = _correlated(n, total, "f32", seed=7200 + n)
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads))
    assert kernels == ["fused_small"], kernels
    ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], dtype="f32", threads=0)
    _check(out, ref, np.array([0, total]), 1e-5)


@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_unaligned_buffers(lib, dtype):
    offsets = workloads.offsets_from_sizes(MIXED)
    total = int(offsets[-1])
    base = _correlated(3, total + 1, dtype, seed=7300)
    grads = [b[1:] if w % 2 == 0 else b[:-1] for w, b in enumerate(base)]
    assert any(g.data_ptr() % 16 for g in grads)
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets))
    assert kernels[0] == "fused_small", kernels
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0)
    _check(out, ref, offsets, TOL[dtype])


@pytest.mark.parametrize("n", [3, 5, 6, 8])
def test_other_orders(lib, n):
    offsets = workloads.offsets_from_sizes(MIXED)
    grads = _correlated(n, int(offsets[-1]), "f32", seed=7400 + n)
    arrays = [_np(g, "f32") for g in grads]
    out, kernels = _kernels(lib, lambda: lib.adasum_reduce(grads, offsets, flags=LINEAR))
    assert kernels[0] == "fused_small", kernels
    _check(out, oracle.adasum_reduce(arrays, offsets=offsets, dtype="f32", linear_order=True, threads=0), offsets, 1e-5)
    out = lib.adasum_reduce(grads, offsets, flags=TOP_DOWN)
    torch.cuda.synchronize()
    _check(out, oracle.adasum_reduce(arrays, offsets=offsets, dtype="f32", top_down=True, threads=0), offsets, 1e-5)


@pytest.mark.parametrize("dtype,out_dtype,n", [("f32", "f32", 2), ("f16", "f16", 4), ("f32", "bf16", 8)])
def test_delta_form_in_place(lib, dtype, out_dtype, n):
    offsets = workloads.offsets_from_sizes(MIXED)
    total = int(offsets[-1])
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7500 + n)
    start = torch.randn(total, generator=gen, device="cuda").to(TORCH_DT[dtype])
    steps = _correlated(n, total, "f32", seed=7600 + n)
    currents = [(start.float() + s).to(TORCH_DT[dtype]) for s in steps]
    ref = oracle.adasum_reduce_delta([_np(c, dtype) for c in currents], _np(start, dtype), offsets=offsets,
                                     dtype=dtype, threads=0)
    s64 = oracle.decode(_np(start, dtype), dtype)
    if out_dtype == dtype:
        params = start.clone()
        out, kernels = _kernels(lib, lambda: lib.adasum_reduce_delta(currents, params, offsets, out=params))
    else:
        out, kernels = _kernels(lib, lambda: lib.adasum_reduce_delta(currents, start, offsets,
                                                                     out_dtype=TORCH_DT[out_dtype]))
    assert kernels[0] == "fused_small", kernels
    eps = {"f32": 2.0 ** -24, "f16": 2.0 ** -11, "bf16": 2.0 ** -8}[out_dtype]
    got = out.double().cpu().numpy()
    for t in range(len(MIXED)):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi > lo:
            bound = TOL[dtype] * np.linalg.norm(ref[lo:hi] - s64[lo:hi]) + 1.01 * eps * np.linalg.norm(ref[lo:hi])
            assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= bound, t
