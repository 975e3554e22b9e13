"""The cache of per-offset-table segment tables: a call keeps the tables it has looked up alive
until its launches are enqueued, whatever else is dropped from the cache meanwhile."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
SIMPLE = 1 << 16
CACHE_TABLES = 256        # the library keeps at most this many tables


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _inputs(n, total, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    return [0.55 * shared + 0.84 * torch.randn(total, generator=gen, device="cuda") for _ in range(n)]


def test_a_call_survives_the_eviction_of_its_own_table(lib):
    """Order that used to free a table in use: a call with the fp32-pipe kernels caches the short
    segment length for X; a default call adds X's other lengths; other offset tables push the first
    one to the front of the cache; the next call on X finds one of its tables and misses another,
    which evicts the least recently used entry while the call is still holding tables."""
    lib.adasum_shutdown()                                   # start from an empty cache
    sizes_x = [70_000, 300, 9000, 129]
    x_off = workloads.offsets_from_sizes(sizes_x)
    grads = _inputs(16, int(x_off[-1]), seed=6000)
    ref = oracle.adasum_reduce([g.cpu().numpy() for g in grads], offsets=x_off, dtype="f32", threads=0)

    def check(out):
        torch.cuda.synchronize()
        got = out.double().cpu().numpy()
        for t in range(len(sizes_x)):
            lo, hi = int(x_off[t]), int(x_off[t + 1])
            assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= 1e-5 * np.linalg.norm(ref[lo:hi]), t

    check(lib.adasum_reduce(grads, x_off, flags=SIMPLE))
    check(lib.adasum_reduce(grads, x_off))
    small = _inputs(2, 4096, seed=6001)
    filler_ref = None
    for k in range(CACHE_TABLES + 40):                      # each call adds at least one table
        off = np.array([0, 100 + k, 4096], dtype=np.int64)
        out = lib.adasum_reduce(small, off, flags=SIMPLE | (1 << 17))
        if k == 0:
            torch.cuda.synchronize()
            filler_ref = oracle.adasum_reduce([g.cpu().numpy() for g in small], offsets=off, dtype="f32", threads=0)
            assert np.linalg.norm(out.double().cpu().numpy() - filler_ref) <= 1e-5 * np.linalg.norm(filler_ref)
        if k % 64 == 0:
            check(lib.adasum_reduce(grads, x_off))          # hits and misses interleaved with the evictions
    check(lib.adasum_reduce(grads, x_off))
    check(lib.adasum_reduce(grads, x_off, flags=SIMPLE))
    check(lib.adasum_reduce(grads, x_off, flags=2 | (2 << 8)))
    lib.adasum_shutdown()
    check(lib.adasum_reduce(grads, x_off))                  # and everything is rebuilt after a shutdown


def test_host_threads_share_the_library(lib):
    """Several host threads reduce at the same time, each on a stream and a workspace of its own and
    with tensor tables of its own: the table cache, the pool of side streams (the buffers have tensors
    of at most 64 elements) and the per-thread error text are shared state."""
    import threading

    results, errors = {}, []

    def worker(k):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for rep in range(12):
                    sizes = [30_000 + 64 * k + rep, 9 + k, 64, 5000 + rep, 1]
                    offsets = workloads.offsets_from_sizes(sizes)
                    grads = _inputs(12 + k, int(offsets[-1]), seed=6100 + 100 * k + rep)
                    out = lib.adasum_reduce(grads, offsets, stream=stream)
                    stream.synchronize()
                    results[(k, rep)] = (out.double().cpu().numpy(), [g.cpu().numpy() for g in grads], offsets)
        except Exception as exc:          # noqa: BLE001
            errors.append((k, repr(exc)))

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert len(results) == 48
    for (k, rep), (got, arrays, offsets) in results.items():
        ref = oracle.adasum_reduce(arrays, offsets=offsets, dtype="f32", threads=0)
        for t in range(len(offsets) - 1):
            lo, hi = int(offsets[t]), int(offsets[t + 1])
            assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= 1e-5 * np.linalg.norm(ref[lo:hi]), (k, rep, t)


@pytest.mark.parametrize("n,flags,total_target,lead", [
    (4, SIMPLE | (1 << 17), 8_600_000, 2_000_000),    # fp32 pipes, segments of 8192: tapered from 7.27 M elements
    (2, 1 << 17, 8_500_000, 4_500_000),               # the pair, separate finish (no single launch)
    (16, 0, 7_900_000, 3_000_000),                    # tensor cores, segments of 8192
])
def test_tapered_tables_cover_every_element_once(lib, n, flags, total_target, lead):
    """Pass-1 tables of buffers that fill the GPU at least three times over are cut with shorter
    segments at both ends.  Tensor boundaries are placed inside every zone (the half-length start,
    the full-length middle, the half- and quarter-length end), with odd sizes so that cuts fall off
    the 64-element grid, and every tensor is compared with the oracle."""
    rng = np.random.default_rng(77 + n)
    sizes = [lead, 65, 1031]
    while sum(sizes) < total_target:
        sizes.append(int(rng.choice([97, 513, 2049, 8191, 16385, 40_001, 150_003, 333_337])))
    order = rng.permutation(len(sizes))
    sizes = [sizes[i] for i in order]
    off = workloads.offsets_from_sizes(sizes)
    grads = _inputs(n, int(off[-1]), seed=6100 + n)
    out = lib.adasum_reduce(grads, off, flags=flags)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce([g.cpu().numpy() for g in grads], offsets=off, dtype="f32", threads=0)
    got = out.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    for t in range(len(sizes)):
        lo, hi = int(off[t]), int(off[t + 1])
        assert np.linalg.norm(got[lo:hi] - ref[lo:hi]) <= 1e-5 * np.linalg.norm(ref[lo:hi]), (t, sizes[t])
