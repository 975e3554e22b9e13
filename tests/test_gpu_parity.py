"""Parity of the CUDA path (called through the C ABI) with the fp64 CPU oracle, element by
element on the same seeded inputs.

Tolerances (relative L2 error ||out - ref|| / ||ref||, per tensor and over the whole buffer):
fp32 inputs 1e-5, fp16 / bf16 inputs 2e-3.  A tensor whose reference is exactly zero must be
exactly zero."""
import numpy as np
import pytest
import torch

from oracle import adasum_oracle as oracle
from paper_2006_02924_b200 import workloads

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-3}
TORCH_DT = workloads.TORCH_DTYPES


@pytest.fixture(scope="module")
def lib():
    from paper_2006_02924_b200 import binding

    return binding


def _to_numpy(t: torch.Tensor, dtype: str) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dtype == "bf16" else t.numpy()


def _oracle(grads, offsets, dtype):
    return oracle.adasum_reduce([_to_numpy(g, dtype) for g in grads], offsets=offsets, dtype=dtype,
                                threads=0)


def _compare(out: np.ndarray, ref: np.ndarray, offsets, tol: float):
    """Returns (global rel-L2, worst per-tensor rel-L2); asserts both against tol, for every tensor
    whatever its length."""
    out = out.astype(np.float64)
    assert np.all(np.isfinite(out))
    worst = 0.0
    for t in range(len(offsets) - 1):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        r, o = ref[lo:hi], out[lo:hi]
        nr = np.linalg.norm(r)
        if nr == 0.0:
            assert not np.any(o), f"tensor {t}: reference is exactly zero, output is not"
            continue
        err = np.linalg.norm(o - r) / nr
        assert err <= tol, f"tensor {t} (len {hi - lo}): rel-L2 {err:.3e} > {tol:.3e}"
        worst = max(worst, err)
    nr = np.linalg.norm(ref)
    glob = np.linalg.norm(out - ref) / nr if nr > 0 else 0.0
    assert glob <= tol, f"global rel-L2 {glob:.3e} > {tol}"
    return glob, worst


def _run_and_check(lib, grads, offsets, dtype, flags=0):
    out = lib.adasum_reduce(grads, offsets, flags=flags)
    torch.cuda.synchronize()
    ref = _oracle(grads, offsets, dtype)
    return _compare(out.cpu().numpy(), ref, offsets, TOL[dtype])


def _correlated(n, total, dtype, seed, rho=0.3, scale=1.0, device="cuda"):
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    shared = torch.randn(total, generator=gen, device=device)
    return [((rho ** 0.5) * shared + ((1 - rho) ** 0.5) * torch.randn(total, generator=gen, device=device))
            .mul_(scale).to(TORCH_DT[dtype]) for _ in range(n)]


# ---- closed forms at the size of the first benchmark configuration ------------------------------

def test_c1_pair_one_million_fp32(lib):
    wl = workloads.generate("c1", device="cuda")
    assert wl.n_workers == 2 and wl.total_elems == 1_000_000
    _run_and_check(lib, wl.grads, wl.offsets, "f32")
    out = lib.adasum_pair(wl.grads[0], wl.grads[1])
    ref = _oracle(wl.grads, wl.offsets, "f32")
    _compare(out.cpu().numpy(), ref, wl.offsets, 1e-5)


def test_closed_forms_one_million(lib):
    n = 1_000_000
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    g = torch.randn(n, generator=gen, device="cuda")
    # orthogonal pair (disjoint supports) -> plain sum, exactly
    a, b = g.clone(), torch.randn(n, generator=gen, device="cuda")
    a[1::2] = 0
    b[0::2] = 0
    out = lib.adasum_pair(a, b)
    assert torch.equal(out, a + b)
    # identical pair -> the input
    out = lib.adasum_pair(g, g.clone())
    assert torch.linalg.norm(out - g) / torch.linalg.norm(g) < 1e-6
    # one zero vector -> the other operand, exactly
    z = torch.zeros_like(g)
    assert torch.equal(lib.adasum_pair(z, g), g)
    assert torch.equal(lib.adasum_pair(g, z), g)
    assert torch.equal(lib.adasum_pair(z, z), z)


# ---- small and awkward shapes ---------------------------------------------------------------------

AWKWARD_SIZES = [1, 3, 7, 8, 9, 0, 1023, 4097, 64, 8191, 8193, 20001, 5]


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 16, 17, 33])
def test_awkward_shapes(lib, dtype, n):
    offsets = workloads.offsets_from_sizes(AWKWARD_SIZES)
    grads = _correlated(n, int(offsets[-1]), dtype, seed=100 + n)
    _run_and_check(lib, grads, offsets, dtype)


SIMPLE = 1 << 16      # ADASUM_FLAG_SIMPLE_KERNELS
SEPARATE = 1 << 17    # ADASUM_FLAG_SEPARATE_FINISH


@pytest.mark.parametrize("first,later,extra", [
    (2, 2, 0), (4, 4, 0), (8, 8, 0), (16, 16, 0), (4, 2, 0), (2, 16, 0), (16, 2, 0), (32, 32, 0), (32, 4, 0),
    (2, 32, 0), (2, 2, SIMPLE), (8, 4, SIMPLE), (16, 16, SIMPLE), (2, 2, SEPARATE), (16, 8, SEPARATE),
    (16, 16, SIMPLE | SEPARATE)])
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_every_radix_gives_the_same_tree(lib, dtype, first, later, extra):
    offsets = workloads.offsets_from_sizes([50_000, 17, 3, 70_001, 64])
    for n in (13, 64, 100):
        grads = _correlated(n, int(offsets[-1]), dtype, seed=200 + n)
        _run_and_check(lib, grads, offsets, dtype, flags=lib.flags_radix(first, later) | extra)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("n", [33, 64, 65, 150])
def test_radix_64_for_16_bit_inputs(lib, dtype, n):
    offsets = workloads.offsets_from_sizes([40_000, 9, 30_011, 1, 64, 5000])
    grads = _correlated(n, int(offsets[-1]), dtype, seed=250 + n)
    assert lib.adasum_plan_info(int(offsets[-1]), 6, n, dtype, lib.flags_radix(64, 0))["radices"][0] == 64
    _run_and_check(lib, grads, offsets, dtype, flags=lib.flags_radix(64, 0))


@pytest.mark.parametrize("dtype,n,first", [("f32", 300, 16), ("f16", 600, 32), ("f32", 520, 2), ("bf16", 257, 8)])
def test_more_operands_than_one_launch_carries(lib, dtype, n, first):
    """A launch carries 256 operand pointers; wider levels are split over several launches."""
    offsets = workloads.offsets_from_sizes([2000, 5, 777, 64])
    grads = _correlated(n, int(offsets[-1]), dtype, seed=280 + n, rho=0.7)
    info = lib.adasum_plan_info(int(offsets[-1]), 4, n, dtype, lib.flags_radix(first, 0))
    assert info["launches"] > len(info["radices"]) + 1      # more than one launch per pass somewhere
    _run_and_check(lib, grads, offsets, dtype, flags=lib.flags_radix(first, 0))


def test_radix_64_is_refused_for_fp32(lib):
    grads = _correlated(64, 1000, "f32", seed=260)
    with pytest.raises(lib.AdasumError):
        lib.adasum_reduce(grads, [0, 1000], flags=lib.flags_radix(64, 0))


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_unaligned_buffers_on_the_tensor_core_path(lib, dtype):
    sizes = [3000, 33, 20_000, 7]
    offsets = workloads.offsets_from_sizes(sizes)
    total = int(offsets[-1])
    base = _correlated(40, total + 1, dtype, seed=270)
    grads = [b[1:] if w % 2 == 0 else b[:-1] for w, b in enumerate(base)]
    assert any(g.data_ptr() % 16 for g in grads)
    for first in (16, 32):
        _run_and_check(lib, grads, offsets, dtype, flags=lib.flags_radix(first, 0))


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_unaligned_buffers_take_the_scalar_path(lib, dtype):
    """Worker buffers that start 1 element into an allocation are not 16-byte aligned."""
    sizes = [1000, 33, 9000, 7]
    offsets = workloads.offsets_from_sizes(sizes)
    total = int(offsets[-1])
    base = _correlated(4, total + 1, dtype, seed=300)
    grads = [b[1:] if w % 2 == 0 else b[:-1] for w, b in enumerate(base)]
    assert any(g.data_ptr() % 16 for g in grads)
    _run_and_check(lib, grads, offsets, dtype)
    out_store = torch.empty(total + 1, device="cuda")
    aligned = [b[:-1].clone() for b in base]
    out = lib.adasum_reduce(aligned, offsets, out=out_store[1:])
    ref = _oracle(aligned, offsets, dtype)
    _compare(out.cpu().numpy(), ref, offsets, TOL[dtype])


def test_single_long_tensor_many_segments(lib):
    offsets = np.array([0, 3_000_001], dtype=np.int64)
    grads = _correlated(4, 3_000_001, "f32", seed=400, scale=1e-3)
    _run_and_check(lib, grads, offsets, "f32")


def test_zero_tensors_inside_a_deep_tree(lib):
    offsets = workloads.offsets_from_sizes([5000, 300, 12000])
    grads = _correlated(32, int(offsets[-1]), "f32", seed=500)
    for w in (0, 1, 2, 3, 5, 8, 13, 21, 30, 31):
        grads[w][5000:5300] = 0
    for w in range(32):
        grads[w][:5000] = 0            # a tensor that is zero on every worker
    for flags in (0, lib.flags_radix(2, 2), lib.flags_radix(4, 8)):
        _run_and_check(lib, grads, offsets, "f32", flags=flags)


def test_fp16_subnormal_magnitudes(lib):
    offsets = workloads.offsets_from_sizes([4096, 10_000])
    grads = _correlated(8, int(offsets[-1]), "f16", seed=600, scale=3e-6)
    assert float(grads[0].float().abs().max()) < 6.2e-5        # all values are fp16 subnormals
    assert float(grads[0].float().abs().max()) > 0
    _run_and_check(lib, grads, offsets, "f16")


def test_results_are_deterministic(lib):
    wl = workloads.generate("c2", device="cuda", tensor_sizes=workloads.reduced_sizes(
        workloads.resnet50_tensor_sizes(), 16))
    first = lib.adasum_reduce(wl.grads, wl.offsets).clone()
    for _ in range(3):
        assert torch.equal(lib.adasum_reduce(wl.grads, wl.offsets), first)


def test_guard_bands_are_untouched(lib):
    """Output and workspace are written only inside their stated extents."""
    offsets = workloads.offsets_from_sizes([777, 12_345, 1])
    total = int(offsets[-1])
    grads = _correlated(20, total, "f32", seed=700)
    need = lib.adasum_workspace_bytes(total, 3, 20, "f32")
    pad = 1024
    store = torch.full((total + 2 * pad,), 12345.0, device="cuda")
    ws = torch.full((need + 2 * 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    out = store[pad:pad + total]
    lib.adasum_reduce(grads, offsets, out=out, workspace=ws[4096:4096 + need])
    torch.cuda.synchronize()
    assert bool((store[:pad] == 12345.0).all()) and bool((store[pad + total:] == 12345.0).all())
    assert bool((ws[:4096] == 0x5A).all()) and bool((ws[4096 + need:] == 0x5A).all())
    _compare(out.cpu().numpy(), _oracle(grads, offsets, "f32"), offsets, 1e-5)


def test_too_small_workspace_is_rejected(lib):
    grads = _correlated(4, 1000, "f32", seed=800)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.AdasumError) as err:
        lib.adasum_reduce(grads, [0, 1000], workspace=ws)
    assert err.value.status == 5


# ---- the benchmark configurations, reduced (whole buffer against the oracle) ----------------------

@pytest.mark.parametrize("name,divisor,n", [("c2", 8, None), ("c3", 256, None), ("c4", 512, None), ("c5", 64, None)])
def test_reduced_configurations(lib, name, divisor, n):
    spec = workloads.SPECS[name]
    sizes = workloads.reduced_sizes(spec.tensor_sizes(), divisor)
    wl = workloads.generate(spec, device="cuda", tensor_sizes=sizes, n_workers=n)
    glob, worst = _run_and_check(lib, wl.grads, wl.offsets, spec.dtype)
    print(f"{name}/{divisor}: global {glob:.2e} worst tensor {worst:.2e}")


# ---- the benchmark configurations at full size ---------------------------------------------------

def test_c2_full_size_every_tensor(lib):
    wl = workloads.generate("c2", device="cuda")
    assert wl.num_tensors == 161 and wl.total_elems == 25_557_032
    glob, worst = _run_and_check(lib, wl.grads, wl.offsets, "f32")
    print(f"c2 full: global {glob:.2e} worst tensor {worst:.2e}")


def test_c2_full_size_literal_tree(lib):
    """The same workload as the level-by-level tree of Algorithm 1 (radix 2 everywhere), where every
    level's combine is fused with the next level's dot products; and the same with separate kernels."""
    wl = workloads.generate("c2", device="cuda")
    for flags in (lib.flags_radix(2, 2), lib.flags_radix(2, 2) | lib.ADASUM_FLAG_NO_LEVEL_FUSION):
        glob, worst = _run_and_check(lib, wl.grads, wl.offsets, "f32", flags=flags)
        print(f"c2 full, literal tree (flags {flags:#x}): global {glob:.2e} worst tensor {worst:.2e}")


def _sampled_tensor_check(lib, name, sample_count, max_len, also=()):
    """Full-size run in the launch configuration the benchmark uses; a sample of tensors (every
    size class up to max_len elements, seeded choice) and the tensors listed in `also` (the largest
    ones: the embedding table and feed-forward matrices) are reduced by the oracle and compared."""
    spec = workloads.SPECS[name]
    wl = workloads.generate(spec, device="cuda")
    out = lib.adasum_reduce(wl.grads, wl.offsets)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out).all())
    sizes = np.diff(wl.offsets)
    rng = np.random.default_rng(workloads.BASE_SEED + spec.seed_index)
    eligible = np.flatnonzero(sizes <= max_len)
    chosen = set(rng.choice(eligible, size=min(sample_count, eligible.size), replace=False).tolist())
    chosen.add(int(eligible[np.argmax(sizes[eligible])]))      # the largest eligible tensor
    chosen.add(int(np.argmin(sizes)))                          # and the smallest
    chosen.update(int(t) for t in wl.zeroed if sizes[t] <= max_len)
    chosen.update(int(t) for t in also)
    chosen = sorted(chosen, key=lambda t: -int(sizes[t]))      # longest first: the oracle's threads take whole tensors
    # one oracle call over the chosen tensors packed side by side (its threads run across tensors)
    packed_offsets = workloads.offsets_from_sizes([int(sizes[t]) for t in chosen])
    packed = [torch.cat([g[int(wl.offsets[t]):int(wl.offsets[t + 1])] for t in chosen]) for g in wl.grads]
    got = torch.cat([out[int(wl.offsets[t]):int(wl.offsets[t + 1])] for t in chosen]).cpu().numpy()
    ref = _oracle(packed, packed_offsets, spec.dtype)
    del packed
    _, worst = _compare(got, ref, packed_offsets, TOL[spec.dtype])
    share = float(sum(int(sizes[t]) for t in chosen)) / float(wl.total_elems)
    print(f"{name} full size: {len(chosen)} tensors checked ({100 * share:.0f} % of the elements, largest "
          f"{int(sizes[chosen[0]])}), worst rel-L2 {worst:.2e}")


# BERT-Large list: tensor 0 is the word-embedding table (31,254,528 elements), 15 + 16 k / 17 + 16 k are
# layer k's feed-forward matrices (4,194,304 elements each)
def test_c3_full_size_sampled_tensors(lib):
    _sampled_tensor_check(lib, "c3", sample_count=24, max_len=4_200_000, also=(0, 15, 17 + 16 * 23))


def test_c4_full_size_sampled_tensors(lib):
    _sampled_tensor_check(lib, "c4", sample_count=20, max_len=1_100_000, also=(0, 15, 17 + 16 * 11, 17 + 16 * 23))


def test_c5_full_size_sampled_tensors(lib):
    _sampled_tensor_check(lib, "c5", sample_count=24, max_len=2_400_000)
