"""adasum_pair_noalloc: the pair operator for hosts that cannot allocate device memory when they
call the library (a memory-pool callback, a process whose GPU budget belongs to another
allocator, a loop that forbids driver allocations after start-up).  The entry point keeps its
scratch in a fixed array inside the library instead of taking a workspace, so the test checks that
it returns what adasum_pair returns, twice in a row with different inputs and tensor tables (the
second call finds the first call's leftovers in the shared scratch), and that it refuses inputs
larger than the fixed scratch can serve.

Collected last on purpose: a failure here cannot hide results of the other GPU tests."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu


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


def _rel(x, y):
    return float(torch.linalg.norm(x.double() - y.double()) / torch.linalg.norm(y.double()))


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.float16, 2e-3)])
def test_two_calls_in_a_row_match_adasum_pair(lib, dtype, tol):
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
        assert bool(torch.isfinite(got).all())
        assert _rel(got, expected) <= tol
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            if hi - lo >= 64:
                assert _rel(got[lo:hi], expected[lo:hi]) <= tol


def test_one_million_elements_like_the_first_benchmark_case(lib):
    wl = workloads.generate("c1", device="cuda")
    expected = lib.adasum_pair(wl.grads[0], wl.grads[1])
    for _ in range(2):
        got = lib.adasum_pair_noalloc(wl.grads[0], wl.grads[1])
        assert _rel(got, expected) <= 1e-5


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
