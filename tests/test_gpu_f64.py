"""GPU parity of the fp64 kernels (Section 4.4: the operator is offered for fp16, fp32 and fp64
tensors) against the fp64 oracle.  Everything on the device is a double, so the bound is a few
hundred ulps of a double, not the fp32 tolerance."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu

TOL = 1e-12
SIZES = [70_001, 0, 33, 4099, 1024, 7, 20_000, 2048, 513]


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _correlated(n, total, seed, rho=0.4):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda", dtype=torch.float64)
    return [(rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device="cuda",
                                                                     dtype=torch.float64) for _ in range(n)]


def _check(out, ref, offsets, tol):
    got = out.double().cpu().numpy()
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


@pytest.mark.parametrize("n,radices", [(1, (0, 0)), (2, (0, 0)), (3, (0, 0)), (4, (0, 0)), (5, (2, 2)), (8, (2, 2)),
                                       (8, (4, 2)), (16, (0, 0)), (37, (0, 0)), (64, (2, 4)), (300, (0, 0)),
                                       (130, (2, 2))])
def test_f64_parity(lib, n, radices):
    offsets = workloads.offsets_from_sizes(SIZES)
    grads = _correlated(n, int(offsets[-1]), seed=5100 + n)
    for g in grads[: n // 2]:
        g[int(offsets[6]):int(offsets[7])] = 0                 # a tensor that is zero on half the workers
    for g in grads:
        g[int(offsets[3]):int(offsets[4])] = 0                 # and one that is zero everywhere
    flags = lib.flags_radix(*radices)
    out = lib.adasum_reduce_delta(grads, None, offsets, out_dtype=torch.float64, flags=flags)
    assert out.dtype == torch.float64
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([g.cpu().numpy() for g in grads], offsets=offsets, dtype="f64", threads=0)
    _check(out, ref, offsets, TOL)
    again = lib.adasum_reduce_delta(grads, None, offsets, out_dtype=torch.float64, flags=flags)
    assert torch.equal(out, again)                                 # deterministic
    single = lib.adasum_reduce(grads, offsets, flags=flags)       # the calls with a float* out store fp32
    assert single.dtype == torch.float32
    _check(single, ref, offsets, 1e-7)


def test_f64_resolves_what_fp32_cannot(lib):
    """Two gradients that differ by one part in 1e10: in fp32 they are identical (result g), in fp64
    the small orthogonal component must come through."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    total = 10_000
    g = torch.randn(total, generator=gen, device="cuda", dtype=torch.float64)
    d = torch.randn(total, generator=gen, device="cuda", dtype=torch.float64)
    d -= (d @ g) / (g @ g) * g                                      # orthogonal to g
    a, b = g, g + 1e-10 * d
    out = lib.adasum_reduce_delta([a, b], None, out_dtype=torch.float64)
    ref = oracle.adasum_reduce([a.cpu().numpy(), b.cpu().numpy()], dtype="f64")
    diff = (out - g).cpu().numpy()
    assert np.linalg.norm(diff) > 0
    assert np.linalg.norm(diff - (ref - g.cpu().numpy())) <= 1e-4 * np.linalg.norm(ref - g.cpu().numpy())


def test_f64_orthogonality_and_pair(lib):
    offsets = workloads.offsets_from_sizes([30_000, 33, 4099])
    grads = _correlated(16, int(offsets[-1]), seed=5200)
    out, ortho = lib.adasum_reduce_ex(grads, offsets)
    _, ref_ortho = oracle.adasum_reduce([g.cpu().numpy() for g in grads], offsets=offsets, dtype="f64",
                                        return_orthogonality=True, threads=0)
    assert np.allclose(ortho.cpu().numpy(), ref_ortho, rtol=1e-6)
    pair = lib.adasum_pair(grads[0], grads[1], offsets)
    ref = oracle.adasum_reduce([grads[0].cpu().numpy(), grads[1].cpu().numpy()], offsets=offsets, dtype="f64")
    _check(pair, ref, offsets, 1e-7)


def test_f64_unaligned_buffers(lib):
    total = 50_001
    base = [torch.randn(total + 1, device="cuda", dtype=torch.float64) for _ in range(6)]
    grads = [b[1:] for b in base]                                   # 8-byte but not 16-byte aligned
    out = lib.adasum_reduce_delta(grads, None, out_dtype=torch.float64)
    ref = oracle.adasum_reduce([g.cpu().numpy() for g in grads], dtype="f64")
    _check(out, ref, np.array([0, total], dtype=np.int64), TOL)


@pytest.mark.parametrize("n,in_place", [(1, False), (2, False), (8, True), (21, False)])
def test_f64_delta_form(lib, n, in_place):
    offsets = workloads.offsets_from_sizes([30_000, 33, 4099, 0, 64])
    total = int(offsets[-1])
    start = torch.randn(total, device="cuda", dtype=torch.float64)
    currents = [start + 1e-3 * g for g in _correlated(n, total, seed=5300 + n)]
    ref = oracle.adasum_reduce_delta([c.cpu().numpy() for c in currents], start.cpu().numpy(), offsets=offsets,
                                     dtype="f64", threads=0)
    step = ref - start.cpu().numpy()
    out = lib.adasum_reduce_delta(currents, start, offsets, out=start if in_place else None, out_dtype=torch.float64)
    assert (out.data_ptr() == start.data_ptr()) == in_place
    err = np.linalg.norm(out.cpu().numpy() - ref)
    assert err <= TOL * np.linalg.norm(step) + 2.0 ** -52 * np.linalg.norm(ref)


def test_f64_refusals(lib):
    grads = [torch.randn(256, device="cuda", dtype=torch.float64) for _ in range(4)]
    for flags in (1 << 18, 1 << 20, 1 << 17, 1 << 16, lib.flags_radix(8, 0), lib.flags_radix(2, 16)):
        with pytest.raises(lib.AdasumError):
            lib.adasum_reduce(grads, flags=flags)
    with pytest.raises(lib.AdasumError):                            # fp64 in, 16-bit out
        lib.adasum_reduce_delta(grads, None, out_dtype=torch.bfloat16)
    with pytest.raises(lib.AdasumError):                            # fp32 in, fp64 out
        lib.adasum_reduce_delta([g.float() for g in grads], None, out_dtype=torch.float64)
    with pytest.raises(lib.AdasumError):
        lib.adasum_pair_noalloc(grads[0], grads[1])


def test_f64_resnet_shaped(lib):
    """Eight fp64 workers on the ResNet-50 tensor list (the second configuration's shapes)."""
    sizes = workloads.resnet50_tensor_sizes()
    offsets = workloads.offsets_from_sizes(sizes)
    grads = _correlated(8, int(offsets[-1]), seed=5400, rho=0.3)
    out = lib.adasum_reduce_delta(grads, None, offsets, out_dtype=torch.float64)
    torch.cuda.synchronize()
    picked = [0, 1, 2, 50, 100, 158, 159, 160]                      # a few tensors through the oracle
    for t in picked:
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        ref = oracle.adasum_reduce([g[lo:hi].cpu().numpy() for g in grads], dtype="f64")
        err = np.linalg.norm(out[lo:hi].cpu().numpy() - ref) / np.linalg.norm(ref)
        assert err <= TOL, (t, err)
