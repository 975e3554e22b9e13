"""GPU parity of the two by-products of the Gram formulation against the fp64 oracle: the
per-tensor orthogonality measure (Section 3.6) and the sequential recursion (Section 3.4)."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu

TORCH_DT = workloads.TORCH_DTYPES
LINEAR = 1 << 18


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _correlated(n, total, dtype, seed, rho=0.5):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [((rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device="cuda"))
            .to(TORCH_DT[dtype]) for _ in range(n)]


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-4), ("f16", 5e-3), ("bf16", 2e-2)])
@pytest.mark.parametrize("n,flags", [(2, 0), (8, 0), (13, 0), (64, 0), (64, (16) | (4 << 8)), (100, (8) | (16 << 8)),
                                      (16, 1 << 17)])
def test_orthogonality_measure(lib, dtype, tol, n, flags):
    offsets = workloads.offsets_from_sizes([30_000, 17, 0, 4099, 64])
    grads = _correlated(n, int(offsets[-1]), dtype, seed=900 + n)
    for g in grads:
        g[30_000:30_017] = 0                       # a tensor that is zero on every worker
    out, ortho = lib.adasum_reduce_ex(grads, offsets, flags=flags)
    torch.cuda.synchronize()
    ref, ref_ortho = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype,
                                          return_orthogonality=True, threads=0)
    got = ortho.cpu().numpy().astype(np.float64)
    assert np.isnan(got[1]) and np.isnan(ref_ortho[1])       # all-zero leaves
    assert np.isnan(got[2])                                  # empty tensor
    for t in (0, 3, 4):
        assert abs(got[t] - ref_ortho[t]) <= tol * ref_ortho[t], (t, got[t], ref_ortho[t])
    assert 1.0 / n - 1e-3 <= got[0] <= 1.0 + 1e-3
    same = lib.adasum_reduce(grads, offsets, flags=flags)
    assert torch.equal(same, out)                           # asking for the measure does not change the result


def test_orthogonality_extremes(lib):
    """Section 3.6: 1 for mutually orthogonal gradients, 1/n for identical ones (n = 64)."""
    n, width = 64, 256
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    ortho_inputs = []
    for w in range(n):
        g = torch.zeros(n * width, device="cuda")
        g[w * width:(w + 1) * width] = (1 + w) * torch.randn(width, generator=gen, device="cuda")
        ortho_inputs.append(g)
    _, measure = lib.adasum_reduce_ex(ortho_inputs)
    assert abs(float(measure[0]) - 1.0) < 1e-5
    g = torch.randn(10_000, generator=gen, device="cuda")
    _, measure = lib.adasum_reduce_ex([g.clone() for _ in range(n)])
    assert abs(float(measure[0]) - 1.0 / n) < 1e-6


def test_orthogonality_needs_two_workers(lib):
    g = torch.randn(100, device="cuda")
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce_ex([g])


@pytest.mark.parametrize("dtype,n,tol", [("f32", 2, 1e-5), ("f32", 3, 1e-5), ("f32", 5, 1e-5), ("f32", 16, 1e-5),
                                         ("f32", 32, 1e-5), ("f16", 7, 2e-3), ("f16", 64, 2e-3), ("bf16", 33, 2e-3)])
def test_linear_order(lib, dtype, n, tol):
    offsets = workloads.offsets_from_sizes([20_000, 33, 4097, 128])
    grads = _correlated(n, int(offsets[-1]), dtype, seed=950 + n, rho=0.6)
    out, ortho = lib.adasum_reduce_ex(grads, offsets, flags=LINEAR)
    torch.cuda.synchronize()
    hosts = [_np(g, dtype) for g in grads]
    ref, ref_ortho = oracle.adasum_reduce(hosts, offsets=offsets, dtype=dtype, linear_order=True,
                                          return_orthogonality=True, threads=0)
    got = out.cpu().numpy().astype(np.float64)
    for t in range(4):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        err = np.linalg.norm(got[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi])
        assert err <= tol, (t, err)
        assert abs(float(ortho[t]) - ref_ortho[t]) <= max(10 * tol, 1e-4) * ref_ortho[t]
    if n > 3:      # for three workers the tree with its carried last operand IS the sequential order
        tree = oracle.adasum_reduce(hosts, offsets=offsets, dtype=dtype, threads=0)
        assert np.linalg.norm(got - tree) / np.linalg.norm(tree) > 10 * tol      # it really is another order


def test_linear_order_limits(lib):
    grads = [torch.randn(64, device="cuda") for _ in range(33)]
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce(grads, flags=LINEAR)
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce(grads[:8], flags=LINEAR | lib.flags_radix(8, 0))


TOP_DOWN = 1 << 20


@pytest.mark.parametrize("dtype,n,tol", [("f32", 3, 1e-5), ("f32", 5, 1e-5), ("f32", 6, 1e-5), ("f32", 7, 1e-5),
                                         ("f32", 13, 1e-5), ("f32", 24, 1e-5), ("f32", 31, 1e-5), ("f16", 11, 2e-3),
                                         ("f16", 48, 2e-3), ("bf16", 63, 2e-3)])
def test_top_down_halves(lib, dtype, n, tol):
    """The tree of Section 3.4 split from the top, for worker counts that are not powers of two."""
    offsets = workloads.offsets_from_sizes([20_000, 33, 4097, 128])
    grads = _correlated(n, int(offsets[-1]), dtype, seed=1950 + n, rho=0.6)
    out, ortho = lib.adasum_reduce_ex(grads, offsets, flags=TOP_DOWN)
    torch.cuda.synchronize()
    hosts = [_np(g, dtype) for g in grads]
    ref, ref_ortho = oracle.adasum_reduce(hosts, offsets=offsets, dtype=dtype, top_down=True,
                                          return_orthogonality=True, threads=0)
    got = out.cpu().numpy().astype(np.float64)
    for t in range(4):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        err = np.linalg.norm(got[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi])
        assert err <= tol, (t, err)
        assert abs(float(ortho[t]) - ref_ortho[t]) <= max(10 * tol, 1e-4) * ref_ortho[t]
    if dtype == "f32":     # the two trees differ by a fraction of a percent: visible above the fp32 tolerance only
        tree = oracle.adasum_reduce(hosts, offsets=offsets, dtype=dtype, threads=0)
        assert np.linalg.norm(got - tree) / np.linalg.norm(tree) > 10 * tol      # it really is another tree


def test_top_down_halves_limits_and_powers_of_two(lib):
    offsets = workloads.offsets_from_sizes([9000, 77])
    grads = _correlated(16, int(offsets[-1]), "f32", seed=1990)
    same = lib.adasum_reduce(grads, offsets, flags=TOP_DOWN)         # a power of two: the same tree, the same plan
    want = lib.adasum_reduce(grads, offsets)
    torch.cuda.synchronize()
    assert torch.equal(same, want)
    big = lib.adasum_reduce(_correlated(128, 4096, "f32", seed=1991), flags=TOP_DOWN)     # 128 = 2^7: allowed
    torch.cuda.synchronize()
    assert bool(torch.isfinite(big).all())
    with pytest.raises(lib.AdasumError):                             # 33 fp32 workers do not fit one level
        lib.adasum_reduce([torch.randn(64, device="cuda") for _ in range(33)], flags=TOP_DOWN)
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce(grads[:6], flags=TOP_DOWN | LINEAR)
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce(grads[:6], flags=TOP_DOWN | lib.flags_radix(8, 0))


def test_reduce_can_be_replayed_from_a_cuda_graph(lib):
    """After one ordinary call (which builds the cached segment tables) the reduce is a fixed
    sequence of stream operations: capture it once, replay it on new data."""
    offsets = workloads.offsets_from_sizes([50_000, 300, 9001])
    total = int(offsets[-1])
    grads = _correlated(20, total, "f32", seed=990)
    out = torch.empty(total, device="cuda")
    ws = torch.empty(lib.adasum_workspace_bytes(total, 3, 20, "f32"), dtype=torch.uint8, device="cuda")
    expected_first = lib.adasum_reduce(grads, offsets, out=out, workspace=ws).clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        lib.adasum_reduce(grads, offsets, out=out, workspace=ws)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, expected_first)
    fresh = _correlated(20, total, "f32", seed=991)
    for dst, src in zip(grads, fresh):
        dst.copy_(src)                                # same buffers, new contents
    graph.replay()
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], offsets=offsets, threads=0)
    got = out.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("n", [64, 128])
def test_radix_64_tensor_memory_kernel(lib, dtype, n):
    """Complete groups of 64 fp16 / bf16 workers go through the tcgen05 kernel: same result as the
    mma.sync kernel (flag bit 19) and as the oracle; no device-side wait ran out."""
    offsets = workloads.offsets_from_sizes([70_000, 9, 4097, 1, 64, 33_000])
    total = int(offsets[-1])
    grads = _correlated(n, total, dtype, seed=1500 + n)
    flags = lib.flags_radix(64, 0)
    need = lib.adasum_workspace_bytes(total, 6, n, dtype, flags)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags)
    assert lib.adasum_device_status(total, 6, n, dtype, ws, flags=flags) == 0
    other = lib.adasum_reduce(grads, offsets, flags=flags | (1 << 19))
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0)
    got = out.cpu().numpy().astype(np.float64)
    for t in (0, 2, 4, 5):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi]) <= 2e-3, t
    assert float(torch.linalg.norm(out - other) / torch.linalg.norm(other)) <= 1e-4


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_gpu_usable(lib):
    """The radix-64 tensor-memory kernel bounds every wait on the tensor core.  With the self-test flag
    it leaves each segment's last tile unmultiplied, so the epilogue's wait for that tile (limit:
    microseconds) runs out with no multiplication outstanding; the kernel records it, frees its tensor
    memory and returns.  The host reads ADASUM_ERR_TIMEOUT, and the next ordinary reduce on the same
    workspace is correct and reads status 0."""
    offsets = workloads.offsets_from_sizes([20_000, 513, 6000])
    total = int(offsets[-1])
    grads = _correlated(64, total, "f16", seed=1800)
    flags = lib.flags_radix(64, 0)
    ws = torch.empty(lib.adasum_workspace_bytes(total, 3, 64, "f16", flags), dtype=torch.uint8, device="cuda")
    good = lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags).clone()
    assert lib.adasum_device_status(total, 3, 64, "f16", ws, flags=flags) == 0
    lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags | lib.ADASUM_FLAG_SELFTEST_TIMEOUT)
    assert lib.adasum_device_status(total, 3, 64, "f16", ws, flags=flags | lib.ADASUM_FLAG_SELFTEST_TIMEOUT) == 7
    assert "bounded wait" in lib.adasum_last_error()
    again = lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags)
    assert lib.adasum_device_status(total, 3, 64, "f16", ws, flags=flags) == 0
    torch.cuda.synchronize()
    assert torch.equal(again, good)
    ref = oracle.adasum_reduce([_np(g, "f16") for g in grads], offsets=offsets, dtype="f16", threads=0)
    assert np.linalg.norm(again.cpu().numpy() - ref) <= 2e-3 * np.linalg.norm(ref)


def _stacked(n, total, dtype, seed, pad=0, rho=0.4):
    """Worker buffers that are rows of one [n, total + pad] allocation (a uniform pitch between them)."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    store = torch.empty((n, total + pad), dtype=TORCH_DT[dtype], device="cuda")
    for w in range(n):
        store[w, :total] = (rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device="cuda")
    return store, [store[w, :total] for w in range(n)]


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("n,sizes,pad", [
    (64, [70_000, 9, 4097, 1, 64, 33_000], 3),          # tensors start anywhere, odd pitch
    (64, [65_536, 1024, 512, 131_072], 0),              # everything on the 64-element grid
    (320, [9000, 130, 64, 20_000], 0)])                 # more than one launch of 256 operands, last one a single group
def test_radix_64_kernel_on_rows_of_one_allocation(lib, dtype, n, sizes, pad):
    """Worker buffers that are rows of one [workers, elements] array (a uniform pitch between them),
    as the synthetic workloads hand them out: segments of 1 to 16 tiles, several groups."""
    offsets = workloads.offsets_from_sizes(sizes)
    total = int(offsets[-1])
    store, grads = _stacked(n, total, dtype, seed=1600 + n + pad, pad=pad)
    flags = lib.flags_radix(64, 0)
    need = lib.adasum_workspace_bytes(total, len(sizes), n, dtype, flags)
    ws = torch.full((need,), 0x5A, dtype=torch.uint8, device="cuda")
    out = lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags)
    assert lib.adasum_device_status(total, len(sizes), n, dtype, ws, flags=flags) == 0
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([_np(g, dtype) for g in grads], offsets=offsets, dtype=dtype, threads=0)
    got = out.cpu().numpy().astype(np.float64)
    for t in range(len(sizes)):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= 2e-3 * np.linalg.norm(ref[lo:hi]), t
    again = lib.adasum_reduce(grads, offsets, workspace=ws, flags=flags)
    assert torch.equal(out, again)


@pytest.mark.parametrize("n,total", [(2, 1_000_000), (8, 300_000), (8, 40_000_000)])
def test_device_status_is_clean_on_a_dirty_workspace(lib, n, total):
    """The workspace arrives with arbitrary contents; after a reduce the status word reads 0, on the
    single-launch path (which clears it in the kernel) as on the two-pass path (cleared by the host)."""
    grads = _correlated(n, total, "f32", seed=1700 + n)
    need = lib.adasum_workspace_bytes(total, 1, n, "f32")
    ws = torch.full((need,), 0xAB, dtype=torch.uint8, device="cuda")
    lib.adasum_profile_enable(16)
    out = lib.adasum_reduce(grads, workspace=ws)
    assert lib.adasum_device_status(total, 1, n, "f32", ws) == 0
    kinds = {r["kernel"] for r in lib.adasum_profile_collect(16)}
    assert ("fused_small" in kinds) == (n * total * 4 <= 96 << 20), kinds
    ref = oracle.adasum_reduce([_np(g, "f32") for g in grads], dtype="f32", threads=0)
    assert np.linalg.norm(out.cpu().numpy() - ref) / np.linalg.norm(ref) <= 1e-5
    again = lib.adasum_reduce(grads, workspace=ws)             # the same workspace a second time
    assert torch.equal(out, again)
