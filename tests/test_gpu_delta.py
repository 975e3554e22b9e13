"""adasum_reduce_delta: out = start + Adasum_w(currents[w] - start) (Section 4.1), and the choice of
output type, against the oracle.

Tolerance.  With r = Adasum(...) the exact combination of the effective gradients, the library
computes r to the usual relative tolerance (1e-5 for fp32 buffers, 2e-3 for fp16 / bf16) and then
stores start + r rounded once to the output type, an error of at most half an ulp of the output
element: 2^-24 |out| for fp32, 2^-11 for fp16, 2^-8 for bf16.  So the bound is

    |out - ref| <= tol * |r| + eps_out * |ref|          (2-norms over a tensor)

and the first term is the one that tests the arithmetic; `step = 1` makes it dominate."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES
TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
EPS_OUT = {"f32": 2.0 ** -24, "f16": 2.0 ** -11, "bf16": 2.0 ** -8}


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _case(n, total, dtype, step, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    start = torch.randn(total, generator=gen, device="cuda").to(TORCH_DT[dtype])
    shared = torch.randn(total, generator=gen, device="cuda")
    currents = [(start.float() + step * (0.6 * shared + 0.8 * torch.randn(total, generator=gen, device="cuda")))
                .to(TORCH_DT[dtype]) for _ in range(n)]
    return start, currents


def _check(got, ref, ref_start, offsets, dtype, out_dtype):
    got = got.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        r = ref[lo:hi] - ref_start[lo:hi]
        bound = TOL[dtype] * np.linalg.norm(r) + EPS_OUT[out_dtype] * np.linalg.norm(ref[lo:hi])
        assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= bound, (t, np.linalg.norm(got[lo:hi] - ref[lo:hi]), bound)


OFFSETS = workloads.offsets_from_sizes([250_000, 40, 0, 70_011, 64, 5, 130_000, 1001])


@pytest.mark.parametrize("dtype,n,flags", [
    ("f32", 2, 0), ("f32", 4, 0), ("f32", 8, 0), ("f32", 16, 0), ("f32", 40, 0), ("f32", 32, 32), ("f32", 12, 1 << 16),
    ("f32", 8, 1 << 17), ("f32", 6, 1 << 18), ("f32", 1, 0), ("f32", 64, 2 | (2 << 8)),
    ("f16", 2, 0), ("f16", 8, 0), ("f16", 32, 0), ("f16", 64, 0), ("f16", 64, 1 << 19), ("f16", 20, 0),
    ("bf16", 16, 0), ("bf16", 64, 0), ("bf16", 3, 0), ("bf16", 1, 0)])
@pytest.mark.parametrize("step", [1.0, 1e-2])
def test_delta_matches_the_oracle(lib, dtype, n, flags, step):
    total = int(OFFSETS[-1])
    start, currents = _case(n, total, dtype, step, seed=3000 + n)
    out = lib.adasum_reduce_delta(currents, start, OFFSETS, flags=flags)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_delta([_np(c, dtype) for c in currents], _np(start, dtype), offsets=OFFSETS,
                                     dtype=dtype, linear_order=bool(flags & (1 << 18)), threads=0)
    _check(out, ref, oracle.decode(_np(start, dtype), dtype), OFFSETS, dtype, "f32")


@pytest.mark.parametrize("dtype,n", [("f32", 2), ("f32", 8), ("f16", 4)])
def test_small_inputs_take_the_single_launch_path(lib, dtype, n):
    offsets = workloads.offsets_from_sizes([90_000, 33, 20_000])
    start, currents = _case(n, int(offsets[-1]), dtype, 1.0, seed=3100 + n)
    info = lib.adasum_plan_info(int(offsets[-1]), 3, n, dtype)
    assert info["launches"] == 1
    out = lib.adasum_reduce_delta(currents, start, offsets)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_delta([_np(c, dtype) for c in currents], _np(start, dtype), offsets=offsets,
                                     dtype=dtype, threads=0)
    _check(out, ref, oracle.decode(_np(start, dtype), dtype), offsets, dtype, "f32")


@pytest.mark.parametrize("dtype,out_dtype,n", [("f32", "bf16", 8), ("f32", "f16", 16), ("f16", "f16", 32),
                                               ("bf16", "bf16", 8), ("f16", "bf16", 2), ("f32", "bf16", 1)])
def test_output_types(lib, dtype, out_dtype, n):
    total = int(OFFSETS[-1])
    start, currents = _case(n, total, dtype, 1.0, seed=3200 + n)
    out = lib.adasum_reduce_delta(currents, start, OFFSETS, out_dtype=TORCH_DT[out_dtype])
    assert out.dtype == TORCH_DT[out_dtype]
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_delta([_np(c, dtype) for c in currents], _np(start, dtype), offsets=OFFSETS,
                                     dtype=dtype, threads=0)
    _check(out, ref, oracle.decode(_np(start, dtype), dtype), OFFSETS, dtype, out_dtype)
    # without a start: the plain reduce, stored in the chosen type
    plain = lib.adasum_reduce_delta(currents, None, OFFSETS, out_dtype=TORCH_DT[out_dtype])
    want = lib.adasum_reduce(currents, OFFSETS)
    torch.cuda.synchronize()
    assert torch.equal(plain, want.to(TORCH_DT[out_dtype]))


@pytest.mark.parametrize("dtype,n", [("f32", 8), ("f32", 40), ("f16", 32), ("f32", 2)])
def test_in_place_update_of_the_parameters(lib, dtype, n):
    total = int(OFFSETS[-1])
    start, currents = _case(n, total, dtype, 1.0, seed=3300 + n)
    want = lib.adasum_reduce_delta(currents, start, OFFSETS, out_dtype=start.dtype)
    params = start.clone()
    got = lib.adasum_reduce_delta(currents, params, OFFSETS, out=params)
    torch.cuda.synchronize()
    assert got.data_ptr() == params.data_ptr()
    assert torch.equal(params, want)


def test_orthogonality_is_that_of_the_effective_gradients(lib):
    total = int(OFFSETS[-1])
    start, currents = _case(8, total, "f32", 1.0, seed=3400)
    ortho = torch.empty(len(OFFSETS) - 1, device="cuda")
    lib.adasum_reduce_delta(currents, start, OFFSETS, orthogonality=ortho)
    torch.cuda.synchronize()
    _, ref = oracle.adasum_reduce_delta([_np(c, "f32") for c in currents], _np(start, "f32"), offsets=OFFSETS,
                                        dtype="f32", return_orthogonality=True, threads=0)
    for t in range(len(OFFSETS) - 1):
        if OFFSETS[t + 1] > OFFSETS[t]:
            assert abs(float(ortho[t]) - ref[t]) <= 1e-4 * ref[t], (t, float(ortho[t]), ref[t])


def test_arguments_are_checked(lib):
    start, currents = _case(4, 4096, "f32", 1.0, seed=3500)
    big = torch.zeros(4096 + 8, device="cuda")
    with pytest.raises(lib.AdasumError):                      # start not 16-byte aligned
        lib.adasum_reduce_delta(currents, big[1:4097], [0, 4096])
    with pytest.raises(lib.AdasumError):                      # a worker's buffer not 16-byte aligned
        lib.adasum_reduce_delta([big[1:4097]] + currents[1:], start, [0, 4096])
    with pytest.raises(lib.AdasumError):                      # out overlaps start but is not start
        both = torch.zeros(8192, device="cuda")
        lib.adasum_reduce_delta(currents, both[:4096], [0, 4096], out=both[4:4100])
    with pytest.raises(lib.AdasumError):                      # start is one of the workers' buffers
        lib.adasum_reduce_delta(currents, currents[2], [0, 4096])
    with pytest.raises(ValueError):
        lib.adasum_reduce_delta(currents, start.half(), [0, 4096])
    torch.cuda.synchronize()


def test_c2_full_size_every_tensor(lib):
    """The benchmark's default workload in the delta form: its gradients are the workers' steps
    from random parameters."""
    wl = workloads.generate("c2", device="cuda")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(3600)
    start = 0.05 * torch.randn(wl.total_elems, generator=gen, device="cuda")
    currents = [start + g for g in wl.grads]
    out = lib.adasum_reduce_delta(currents, start, wl.offsets)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_delta([_np(c, "f32") for c in currents], _np(start, "f32"), offsets=wl.offsets,
                                     dtype="f32", threads=0)
    _check(out, ref, start.double().cpu().numpy(), wl.offsets, "f32", "f32")
