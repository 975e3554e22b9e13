"""adasum_pair_noalloc: the pair operator for hosts that cannot allocate device memory when they
call the library (a memory-pool callback, a process whose GPU budget belongs to another
allocator, a loop that forbids driver allocations after start-up).  The entry point keeps its
scratch in a fixed array inside the library instead of taking a workspace.  The tests check its
result against the fp64 oracle and against adasum_pair, twice in a row with different inputs and
tensor tables (the second call finds the first call's leftovers in the shared scratch), that the
calls leave the amount of free device memory unchanged, and that inputs larger than the fixed
scratch can serve, or a stream that is being captured, are refused.

Collected last on purpose: a failure here cannot hide results of the other GPU tests."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TOL = {torch.float32: 1e-5, torch.float16: 2e-3, torch.bfloat16: 2e-3}
NAME = {torch.float32: "f32", torch.float16: "f16", torch.bfloat16: "bf16"}


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _pair(total, dtype, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    make = lambda: (0.6 * shared + 0.8 * torch.randn(total, generator=gen, device="cuda")).to(dtype)
    return make(), make()


def _np(t):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if t.dtype == torch.bfloat16 else t.numpy()


def _rel(x, y):
    return float(torch.linalg.norm(x.double() - y.double()) / torch.linalg.norm(y.double()))


def _check_against_oracle(got, a, b, offsets, tol):
    ref = oracle.adasum_pair(_np(a), _np(b), offsets=offsets, dtype=NAME[a.dtype])
    out = got.double().cpu().numpy()
    assert np.all(np.isfinite(out))
    for t in range(len(offsets) - 1):               # every tensor, whatever its length
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi > lo:
            err = np.linalg.norm(out[lo:hi] - ref[lo:hi]) / np.linalg.norm(ref[lo:hi])
            assert err <= tol, f"tensor {t} (len {hi - lo}): rel-L2 {err:.3e} > {tol:.1e}"
    assert np.linalg.norm(out - ref) <= tol * np.linalg.norm(ref)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
def test_two_calls_in_a_row_match_the_oracle_and_adasum_pair(lib, dtype):
    tol = TOL[dtype]
    cases = [
        (workloads.offsets_from_sizes([100_003, 7, 64, 250_000, 1]), 11),
        (workloads.offsets_from_sizes([9, 30_001, 5]), 12),      # smaller table: stale entries remain behind it
    ]
    for offsets, seed in cases:
        a, b = _pair(int(offsets[-1]), dtype, seed)
        expected = lib.adasum_pair(a, b, offsets)
        out = torch.full_like(expected, float("nan"))
        got = lib.adasum_pair_noalloc(a, b, offsets, out=out)
        torch.cuda.synchronize()
        assert got.data_ptr() == out.data_ptr()
        _check_against_oracle(got, a, b, offsets, tol)
        assert _rel(got, expected) <= tol


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
def test_buffers_that_are_not_16_byte_aligned(lib, dtype):
    offsets = workloads.offsets_from_sizes([20_001, 3, 4099, 64])
    total = int(offsets[-1])
    a_store, b_store = _pair(total + 1, dtype, 13)
    a, b = a_store[1:], b_store[:-1]
    assert a.data_ptr() % 16 != 0
    out_store = torch.full((total + 1,), float("nan"), device="cuda")
    for _ in range(2):
        got = lib.adasum_pair_noalloc(a, b, offsets, out=out_store[1:])
        torch.cuda.synchronize()
        _check_against_oracle(got, a, b, offsets, TOL[dtype])


def test_the_calls_allocate_no_device_memory(lib):
    """Free device memory (the driver's figure, which sees every allocation of the process) and
    torch's own counters are the same before and after calls that are given their output buffer."""
    offsets = workloads.offsets_from_sizes([300_000, 17, 64, 90_001])
    a, b = _pair(int(offsets[-1]), torch.float32, 14)
    out = torch.empty(int(offsets[-1]), device="cuda")
    lib.adasum_pair_noalloc(a, b, offsets, out=out)              # first call on this device: looks up the scratch address
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    allocated_before, reserved_before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    other = workloads.offsets_from_sizes([5, 200_000, 190_077])   # a tensor table the library has never seen
    assert int(other[-1]) == int(offsets[-1])
    for offs in (offsets, other, offsets):
        lib.adasum_pair_noalloc(a, b, offs, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.cuda.memory_allocated() == allocated_before
        assert torch.cuda.memory_reserved() == reserved_before
    _check_against_oracle(out, a, b, offsets, 1e-5)


def test_a_capturing_stream_is_refused(lib):
    """The call uploads its table from temporary host memory, which a replayed graph would read
    after it is gone; it therefore declines to be recorded and records nothing."""
    a, b = _pair(50_000, torch.float32, 15)
    out = torch.empty(50_000, device="cuda")
    lib.adasum_pair_noalloc(a, b, out=out)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        graph.capture_begin()
        try:
            with pytest.raises(lib.AdasumError) as err:
                lib.adasum_pair_noalloc(a, b, out=out, stream=stream)
            assert err.value.status == 2 and "CUDA graph" in str(err.value)
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    got = lib.adasum_pair_noalloc(a, b, out=out)                 # and the library still works afterwards
    torch.cuda.synchronize()
    _check_against_oracle(got, a, b, np.array([0, 50_000]), 1e-5)


def test_one_million_elements_like_the_first_benchmark_case(lib):
    wl = workloads.generate("c1", device="cuda")
    expected = lib.adasum_pair(wl.grads[0], wl.grads[1])
    for _ in range(2):
        got = lib.adasum_pair_noalloc(wl.grads[0], wl.grads[1])
        torch.cuda.synchronize()
        assert _rel(got, expected) <= 1e-5
        _check_against_oracle(got, wl.grads[0], wl.grads[1], wl.offsets, 1e-5)


def test_sizes_beyond_the_fixed_scratch_are_refused(lib):
    """Only the host-side checks run: the device pointers are never dereferenced."""
    raw = lib.raw()
    too_many = np.array([0, lib.ADASUM_NOALLOC_MAX_ELEMS + 1], dtype=np.int64)
    status = raw.adasum_pair_noalloc(0x10000000, 0x50000000, too_many.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                                     1, 0, 0x90000000, None)
    assert lib.adasum_status_string(status) == "ADASUM_ERR_ARG"
    assert "static scratch" in lib.adasum_last_error()
    many = np.zeros(lib.ADASUM_NOALLOC_MAX_TENSORS + 2, dtype=np.int64)
    status = raw.adasum_pair_noalloc(0x10000000, 0x50000000, many.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                                     lib.ADASUM_NOALLOC_MAX_TENSORS + 1, 0, 0x90000000, None)
    assert lib.adasum_status_string(status) == "ADASUM_ERR_ARG"
    assert "static scratch" in lib.adasum_last_error()
