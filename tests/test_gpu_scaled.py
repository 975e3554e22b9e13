"""adasum_reduce_scaled (dynamic scaling, Section 4.4.1): the buffers hold scale x gradient, the
result is the operator applied to the gradients themselves.  Against the oracle, which divides
every stored value by its scale in fp64 and runs the plain tree.

Tolerance: that of the plain reduce (relative 2-norm per tensor, 1e-5 for fp32 buffers, 2e-3 for
fp16 / bf16).  The scales enter in fp64 in the coefficient step only, and dividing row i and column
i of a Gram matrix by a worker's scale leaves every entry's relative error what it was."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu
TORCH_DT = workloads.TORCH_DTYPES
TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
SIMPLE, SEPARATE, LINEAR, TOP_DOWN, NO_TC = 1 << 16, 1 << 17, 1 << 18, 1 << 20, 1 << 19


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _np(t, dtype):
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _case(n, offsets, dtype, seed, spread=6.0):
    """True gradients with a common component; scales 2^u, u uniform in [-spread, spread], one per
    (worker, tensor), not powers of two; the stored buffers are gradient x scale rounded to dtype."""
    total = int(offsets[-1])
    num_tensors = len(offsets) - 1
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device="cuda")
    scales = torch.exp2((torch.rand(n, num_tensors, generator=gen, device="cuda") * 2 - 1) * spread).contiguous()
    lengths = torch.tensor(np.diff(np.asarray(offsets)), device="cuda")
    stored = []
    for w in range(n):
        g = 0.55 * shared + 0.84 * torch.randn(total, generator=gen, device="cuda")
        per_elem = torch.repeat_interleave(scales[w], lengths)
        stored.append((g * per_elem).to(TORCH_DT[dtype]))
    return stored, scales


def _check(got, ref, offsets, tol):
    got = got.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi > lo:
            err = np.linalg.norm(got[lo:hi] - ref[lo:hi])
            assert err <= tol * np.linalg.norm(ref[lo:hi]), (t, hi - lo, err / np.linalg.norm(ref[lo:hi]))


OFFSETS = workloads.offsets_from_sizes([250_000, 40, 0, 70_011, 64, 5, 1, 130_000, 1001, 2])


PLANS = [(2, 0), (3, 0), (4, SIMPLE), (8, 0), (8, SIMPLE), (12, 0), (16, 0), (16, SEPARATE), (32, 0), (40, 0),
         (64, 0), (64, NO_TC), (7, LINEAR), (11, TOP_DOWN), (16, 2 | (2 << 8)), (16, 4 | (4 << 8))]
# (the last flag only changes what 16-bit inputs do)
CASES = [(d, n, f) for d in ("f32", "f16", "bf16") for n, f in PLANS if not (d == "f32" and f == NO_TC)]


@pytest.mark.parametrize("dtype,n,flags", CASES)
def test_scaled_reduce_matches_the_oracle(lib, dtype, n, flags):
    stored, scales = _case(n, OFFSETS, dtype, seed=9000 + n + (flags >> 8))
    out, ortho = lib.adasum_reduce_scaled(stored, scales, OFFSETS, flags=flags, want_orthogonality=True)
    torch.cuda.synchronize()
    ref, ref_ortho = oracle.adasum_reduce_scaled([_np(s, dtype) for s in stored], scales.cpu().numpy(), offsets=OFFSETS,
                                                 dtype=dtype, linear_order=bool(flags & LINEAR),
                                                 top_down=bool(flags & TOP_DOWN), return_orthogonality=True,
                                                 threads=0)
    _check(out, ref, OFFSETS, TOL[dtype])
    got_ortho = ortho.double().cpu().numpy()
    lens = np.diff(OFFSETS)
    np.testing.assert_allclose(got_ortho[lens > 0], ref_ortho[lens > 0], rtol=20 * TOL[dtype])
    assert np.all(np.isnan(got_ortho[lens == 0]))


@pytest.mark.parametrize("n,dtype", [(2, "f16"), (4, "f32"), (8, "bf16")])
def test_scaled_small_inputs_take_the_single_launch(lib, n, dtype):
    """Up to 8 workers and operands that fit the L2: one cooperative launch, which reads the scales in
    its three coefficient steps (segments, one-warp tensors, tensors of at most 64 elements)."""
    stored, scales = _case(n, OFFSETS, dtype, seed=9500 + n)
    lib.adasum_profile_enable(16)
    out, ortho = lib.adasum_reduce_scaled(stored, scales, OFFSETS, want_orthogonality=True)
    torch.cuda.synchronize()
    assert [r["kernel"] for r in lib.adasum_profile_collect(16)] == ["fused_small"]
    ref, ref_ortho = oracle.adasum_reduce_scaled([_np(s, dtype) for s in stored], scales.cpu().numpy(), offsets=OFFSETS,
                                                 dtype=dtype, return_orthogonality=True, threads=0)
    _check(out, ref, OFFSETS, TOL[dtype])
    lens = np.diff(OFFSETS)
    np.testing.assert_allclose(ortho.double().cpu().numpy()[lens > 0], ref_ortho[lens > 0], rtol=20 * TOL[dtype])


def test_scaled_reduce_differs_from_the_reduce_of_the_stored_values(lib):
    """The test above would also pass if the scales were ignored and the inputs happened to be
    insensitive to them; they are not: the plain reduce of the same buffers is far from the oracle."""
    stored, scales = _case(8, OFFSETS, "f32", seed=9100)
    plain = lib.adasum_reduce(stored, OFFSETS)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_scaled([_np(s, "f32") for s in stored], scales.cpu().numpy(), offsets=OFFSETS,
                                      dtype="f32", threads=0)
    got = plain.double().cpu().numpy()
    assert np.linalg.norm(got - ref) > 0.1 * np.linalg.norm(ref)


def test_unit_scales_give_the_plain_reduce_bit_for_bit(lib):
    """Scales of exactly 1 change no bit, on the two-pass path (flag bit 17) and in the single launch."""
    stored, _ = _case(8, OFFSETS, "f32", seed=9200, spread=0.0)
    ones = torch.ones(8, len(OFFSETS) - 1, device="cuda")
    for flags in (SEPARATE, 0):
        a = lib.adasum_reduce_scaled(stored, ones, OFFSETS, flags=flags)
        b = lib.adasum_reduce(stored, OFFSETS, flags=flags)
        torch.cuda.synchronize()
        assert torch.equal(a, b), flags


@pytest.mark.parametrize("n", [300, 513])
def test_scaled_short_tensors_with_more_workers_than_one_launch(lib, n):
    """More than 256 workers: the tensors of at most 64 elements are reduced in several launches,
    each of which must look up ITS workers' scales."""
    offsets = workloads.offsets_from_sizes([3, 64, 1, 5000, 17])
    stored, scales = _case(n, offsets, "f32", seed=9300 + n, spread=4.0)
    out = lib.adasum_reduce_scaled(stored, scales, offsets)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_scaled([_np(s, "f32") for s in stored], scales.cpu().numpy(), offsets=offsets,
                                      dtype="f32", threads=0)
    _check(out, ref, offsets, TOL["f32"])


def test_small_fp16_gradients_survive_through_their_scale(lib):
    """What the scale is for: gradients of size 1e-7 are below fp16's smallest subnormal (6e-8 spacing)
    and would be stored as zeros or one-bit values; stored with a scale of 2^24 they keep 11 bits,
    and the result, in fp32 and in the gradients' own units, matches the oracle."""
    offsets = workloads.offsets_from_sizes([100_000, 33, 4096])
    total = int(offsets[-1])
    gen = torch.Generator(device="cuda")
    gen.manual_seed(9400)
    shared = torch.randn(total, generator=gen, device="cuda")
    n = 16
    scales = torch.full((n, 3), 2.0 ** 24, device="cuda")
    true = [1e-7 * (0.55 * shared + 0.84 * torch.randn(total, generator=gen, device="cuda")) for _ in range(n)]
    stored = [(g * 2.0 ** 24).to(torch.float16) for g in true]
    out = lib.adasum_reduce_scaled(stored, scales, offsets)
    torch.cuda.synchronize()
    ref = oracle.adasum_reduce_scaled([_np(s, "f16") for s in stored], scales.cpu().numpy(), offsets=offsets,
                                      dtype="f16", threads=0)
    _check(out, ref, offsets, TOL["f16"])
    assert 1e-8 < float(out.abs().max()) < 1e-5
