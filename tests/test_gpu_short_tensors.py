"""Tensors of at most 64 elements against the fp64 oracle at the plain tolerance.

Their result can be a small difference of large terms: for one-element tensors the operator is the
mean of its two operands, so workers that disagree in sign cancel level after level.  fp32 products,
weights and sums lose what cancels; the library therefore reduces such tensors in fp64 from the
loads to the store.  The inputs here are made to cancel on purpose (conditioning of 1e3 and more),
which the general fp32 path would miss at 1e-5."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES
TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
LINEAR, TOP_DOWN, SEPARATE = 1 << 18, 1 << 20, 1 << 17

# short tensors of every kind between long ones: 1, 2, 3 elements, odd lengths, exactly 64, and 65
# (the first length that takes the general path)
SIZES = [1, 5000, 2, 3, 0, 64, 17, 65, 33, 1, 9001, 63]
# The operator is discontinuous where an operand is exactly zero (Adasum(0, b) = b, but Adasum(e, b)
# for a one-element tensor is (e + b) / 2 however small e is).  16-bit values are coarse enough that
# sums of a few one-element leaves hit zero exactly now and then, and whether an fp64 evaluation
# then lands on zero or one rounding error beside it is luck, for the oracle as for the kernel.
# Vectors do not tie by accident, so the 16-bit cases use two elements where fp32 uses one.
SIZES_16 = [2 if s == 1 else s for s in SIZES]


def _sizes(dtype):
    return SIZES if dtype == "f32" else SIZES_16


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _cancelling(n, offsets, dtype, seed, spread=None):
    """Workers whose short tensors nearly cancel: worker w holds sign_w * (base + small noise), signs
    alternating, so that every pair of the first level leaves about a thousandth of its operands.
    Long tensors are ordinary correlated noise."""
    if spread is None:          # a few units in the last place of the 16-bit types would round away
        spread = {"f32": 2e-3, "f16": 2e-2, "bf16": 0.1}[dtype]
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    total = int(offsets[-1])
    base = torch.randn(total, generator=gen, device="cuda")
    base = torch.where(base.abs() < 0.25, torch.full_like(base, 0.5), base)
    short = torch.zeros(total, dtype=torch.bool, device="cuda")
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi - lo <= 64:
            short[lo:hi] = True
    grads = []
    for w in range(n):
        noise = torch.randn(total, generator=gen, device="cuda")
        sign = 1.0 if w % 2 == 0 else -1.0
        cancelling = sign * base * (1.0 + spread * noise)
        ordinary = 0.55 * base + 0.84 * noise
        grads.append(torch.where(short, cancelling, ordinary).to(TORCH_DT[dtype]))
    return grads


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


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", [2, 3, 5, 8, 16, 17, 64, 65, 100, 128, 129, 256])
def test_cancelling_short_tensors(lib, dtype, n):
    offsets = workloads.offsets_from_sizes(_sizes(dtype))
    grads = _cancelling(n, offsets, dtype, seed=5000 + n)
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0)
    # the inputs do cancel: some short tensor's result is far smaller than its leaves
    lo, hi = int(offsets[0]), int(offsets[1])
    if dtype == "f32" and n & (n - 1) == 0:
        assert np.linalg.norm(ref[lo:hi]) < 0.05 * float(grads[0][lo:hi].double().norm())
    out = lib.adasum_reduce(grads, offsets)
    torch.cuda.synchronize()
    _check(out, ref, offsets, TOL[dtype])


@pytest.mark.parametrize("dtype,n", [("f32", 257), ("f32", 300), ("f16", 520), ("bf16", 1000)])
def test_more_workers_than_one_launch_carries(lib, dtype, n):
    """Above 256 workers every launch reduces the sub-tree of its 256 workers to an fp64 vector and
    a last launch reduces those."""
    offsets = workloads.offsets_from_sizes([7, 300, 64, 1 if dtype == "f32" else 2, 0, 40])
    grads = _cancelling(n, offsets, dtype, seed=5100 + n)
    ref, ref_ortho = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0,
                                          return_orthogonality=True)
    out, ortho = lib.adasum_reduce_ex(grads, offsets)
    torch.cuda.synchronize()
    _check(out, ref, offsets, TOL[dtype])
    got = ortho.double().cpu().numpy()
    for t in (0, 2, 3, 5):
        assert abs(got[t] - ref_ortho[t]) <= 1e-6 * ref_ortho[t], (t, got[t], ref_ortho[t])


@pytest.mark.parametrize("flags", [0, 2 | (2 << 8), 4 | (8 << 8), 16 | (16 << 8), SEPARATE, 32 | SEPARATE])
def test_every_plan_leaves_short_tensors_to_the_fp64_kernel(lib, flags):
    offsets = workloads.offsets_from_sizes(SIZES)
    grads = _cancelling(48, offsets, "f32", seed=5200)
    ref, ref_ortho = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32", threads=0,
                                          return_orthogonality=True)
    out, ortho = lib.adasum_reduce_ex(grads, offsets, flags=flags)
    torch.cuda.synchronize()
    _check(out, ref, offsets, 1e-5)
    got = ortho.double().cpu().numpy()
    for t, size in enumerate(SIZES):
        if size == 0:
            assert np.isnan(got[t])
        elif size <= 64:
            assert abs(got[t] - ref_ortho[t]) <= 1e-6 * ref_ortho[t], (t, got[t], ref_ortho[t])
        else:
            assert abs(got[t] - ref_ortho[t]) <= 1e-4 * ref_ortho[t], (t, got[t], ref_ortho[t])


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("n", [2, 5, 6, 7, 11, 24, 32])
def test_other_orders(lib, dtype, n):
    """The sequential recursion and the top-down halves of Section 3.4 on the same inputs."""
    offsets = workloads.offsets_from_sizes(_sizes(dtype))
    grads = _cancelling(n, offsets, dtype, seed=5300 + n)
    arrays = [_np(g, dtype) for g in grads]
    out = lib.adasum_reduce(grads, offsets, flags=LINEAR)
    torch.cuda.synchronize()
    _check(out, oracle.adasum_reduce(arrays, offsets=offsets, dtype=dtype, linear_order=True, threads=0), offsets,
           TOL[dtype])
    out = lib.adasum_reduce(grads, offsets, flags=TOP_DOWN)
    torch.cuda.synchronize()
    _check(out, oracle.adasum_reduce(arrays, offsets=offsets, dtype=dtype, top_down=True, threads=0), offsets,
           TOL[dtype])


@pytest.mark.parametrize("dtype,out_dtype", [("f32", "f32"), ("f16", "f16"), ("f32", "bf16")])
def test_delta_form(lib, dtype, out_dtype):
    """out = start + Adasum(current - start): the short tensors' differences cancel."""
    sizes = _sizes(dtype)
    offsets = workloads.offsets_from_sizes(sizes)
    total = int(offsets[-1])
    steps = _cancelling(12, offsets, "f32", seed=5400, spread={"f32": 2e-3, "f16": 2e-2}[dtype])
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5401)
    start = torch.randn(total, generator=gen, device="cuda").to(TORCH_DT[dtype])
    currents = [(start.float() + 0.5 * s).to(TORCH_DT[dtype]) for s in steps]
    out = lib.adasum_reduce_delta(currents, start, offsets, out_dtype=TORCH_DT[out_dtype])
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_delta([_np(c, dtype) for c in currents], _np(start, dtype), offsets=offsets,
                                     dtype=dtype, threads=0)
    s64 = oracle.decode(_np(start, dtype), dtype)
    eps = {"f32": 2.0 ** -24, "f16": 2.0 ** -11, "bf16": 2.0 ** -8}[out_dtype]
    got = out.double().cpu().numpy()
    for t in range(len(sizes)):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        bound = TOL[dtype] * np.linalg.norm(ref[lo:hi] - s64[lo:hi]) + 1.01 * eps * np.linalg.norm(ref[lo:hi])
        assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= bound, t


def test_a_buffer_of_short_tensors_only(lib):
    sizes = [3, 0, 64, 1, 1, 20, 0]
    offsets = workloads.offsets_from_sizes(sizes)
    for n in (2, 9, 64):
        grads = _cancelling(n, offsets, "f32", seed=5500 + n)
        out, kernels = None, None
        lib.adasum_profile_enable(64)
        out = lib.adasum_reduce(grads, offsets)
        torch.cuda.synchronize()
        kernels = [r["kernel"] for r in lib.adasum_profile_collect(64)]
        assert kernels == ["short_tensors"], kernels
        ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32", threads=0)
        _check(out, ref, offsets, 1e-5)
    pair = lib.adasum_pair(grads[0], grads[1], offsets)
    torch.cuda.synchronize()
    _check(pair, oracle.adasum_pair(_np(grads[0], "f32"), _np(grads[1], "f32"), offsets=offsets), offsets, 1e-5)


def test_unaligned_buffers_and_zero_leaves(lib):
    offsets = workloads.offsets_from_sizes(SIZES_16)
    total = int(offsets[-1])
    base = _cancelling(10, workloads.offsets_from_sizes(SIZES_16 + [1]), "f16", seed=5600)
    grads = [b[1:] if w % 2 == 0 else b[:-1] for w, b in enumerate(base)]
    assert any(g.data_ptr() % 16 for g in grads) and grads[0].numel() == total
    lo, hi = int(offsets[5]), int(offsets[6])
    for w in (0, 1, 4, 9):
        grads[w][lo:hi] = 0                                     # zero leaves inside the tree
    lo1, hi1 = int(offsets[8]), int(offsets[9])
    for g in grads:
        g[lo1:hi1] = 0                                          # a short tensor that is zero everywhere
    out = lib.adasum_reduce(grads, offsets)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([_np(g, "f16") for g in grads], offsets=offsets, dtype="f16", threads=0)
    _check(out, ref, offsets, 2e-3)
    assert not out[lo1:hi1].any()


def test_side_stream_under_graph_capture_and_back_to_back_calls(lib):
    """Outside the per-launch timing mode the fp64 kernel runs on a stream of the library's own, forked
    from the caller's stream and joined to it with events.  Back-to-back calls on one workspace and a
    captured, replayed call must order it correctly against everything else."""
    offsets = workloads.offsets_from_sizes(SIZES)
    total = int(offsets[-1])
    n = 24
    grads = _cancelling(n, offsets, "f32", seed=5700)
    ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32", threads=0)
    out = torch.empty(total, device="cuda")
    ws = torch.empty(lib.adasum_workspace_bytes(total, len(SIZES), n, "f32"), dtype=torch.uint8, device="cuda")
    for _ in range(5):                          # no synchronisation in between
        out.fill_(float("nan"))
        lib.adasum_reduce(grads, offsets, out=out, workspace=ws)
    torch.cuda.synchronize()
    _check(out, ref, offsets, 1e-5)
    side = torch.cuda.Stream()                  # a caller's stream other than the default one
    with torch.cuda.stream(side):
        out.fill_(float("nan"))
        lib.adasum_reduce(grads, offsets, out=out, workspace=ws, stream=side)
        first = out.clone()
    side.synchronize()
    _check(first, ref, offsets, 1e-5)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        lib.adasum_reduce(grads, offsets, out=out, workspace=ws)
    out.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    _check(out, ref, offsets, 1e-5)
    fresh = _cancelling(n, offsets, "f32", seed=5701)
    for dst, src in zip(grads, fresh):
        dst.copy_(src)
    graph.replay()
    torch.cuda.synchronize()
    _check(out, oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, dtype="f32", threads=0), offsets,
           1e-5)
