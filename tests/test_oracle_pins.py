"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix, checked without going
through the oracle's own formula.  Each test names the passage it rests on."""
import math
import os

import numpy as np
import pytest

from oracle import adasum_oracle as oracle
from tree_algebra import leaf_weights_from_gram

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                key, val = line.split()
                vals[key] = float(val)
    return vals


def _rng(seed):
    return np.random.default_rng(seed)


def _rel(x, y):
    return np.linalg.norm(x - y) / max(np.linalg.norm(y), 1e-300)


# -- Section 3.5 (properties): orthogonal operands are summed ---------------------------------
@pytest.mark.parametrize("n", [2, 17, 1000])
def test_orthogonal_pair_is_plain_sum(n):
    rng = _rng(1)
    a = np.zeros(2 * n)
    b = np.zeros(2 * n)
    a[0::2] = rng.standard_normal(n)       # disjoint supports: a.b == 0 exactly
    b[1::2] = 3.0 * rng.standard_normal(n)
    out = oracle.adasum_pair(a, b)
    np.testing.assert_allclose(out, a + b, rtol=0, atol=1e-15)


# -- Section 3.5: parallel operands are averaged; closed form Adasum(g, c g) = (1+c)/2 g -------
@pytest.mark.parametrize("c", [1.0, 2.0, 0.5, -1.0, -3.0, 1e-3])
def test_parallel_pair_closed_form(c):
    g = _rng(2).standard_normal(257)
    out = oracle.adasum_pair(g, c * g)
    np.testing.assert_allclose(out, 0.5 * (1.0 + c) * g, rtol=1e-13, atol=1e-15)


def test_identical_pair_returns_the_input():
    g = _rng(3).standard_normal(1000).astype(np.float32)
    out = oracle.adasum_pair(g, g.copy())
    np.testing.assert_allclose(out, g.astype(np.float64), rtol=1e-14)


# -- Section 3 (operator is symmetric in its arguments; the coefficients swap) ----------------
def test_swap_symmetry_and_coefficient_swap():
    rng = _rng(4)
    a, b = rng.standard_normal(333), 0.2 * rng.standard_normal(333) + 0.1
    np.testing.assert_allclose(oracle.adasum_pair(a, b), oracle.adasum_pair(b, a), rtol=1e-14)
    d, na, nb = float(a @ b), float(a @ a), float(b @ b)
    ca, cb = oracle.coefficients(d, na, nb)
    cb2, ca2 = oracle.coefficients(d, nb, na)
    assert (ca, cb) == (ca2, cb2)
    assert ca != cb                               # a transposed norm would show here


# -- Section 3.3: the operator is the mean of the two one-order sequential emulations ---------
def test_mean_of_both_visiting_orders():
    rng = _rng(5)
    a, b = rng.standard_normal(64), rng.standard_normal(64) + 0.5
    d, na, nb = a @ b, a @ a, b @ b
    order_12 = a + (1.0 - d / nb) * b             # Eq. for w_{1,2}
    order_21 = b + (1.0 - d / na) * a             # Eq. for w_{2,1}
    np.testing.assert_allclose(oracle.adasum_pair(a, b), 0.5 * (order_12 + order_21), rtol=1e-13)


# -- Appendix A.3: matrix form (I - a a^T / 2|a|^2) b + (I - b b^T / 2|b|^2) a ----------------
@pytest.mark.parametrize("n", [1, 2, 5, 16])
def test_matrix_form(n):
    rng = _rng(6 + n)
    a, b = rng.standard_normal(n), rng.standard_normal(n)
    eye = np.eye(n)
    ref = (eye - np.outer(a, a) / (2 * (a @ a))) @ b + (eye - np.outer(b, b) / (2 * (b @ b))) @ a
    np.testing.assert_allclose(oracle.adasum_pair(a, b), ref, rtol=1e-12, atol=1e-14)


# -- Appendix A.3, Lemma (angle): min cos(eta) = 0.9428 at cos^2(gamma) = 2/3 ------------------
def test_lemma_angle_value_from_paper():
    golden = _golden("lemma_angle.txt")
    r = np.array([1.0, 0.0])
    worst, worst_gamma = 1.0, None
    for gamma in np.linspace(0.0, math.pi / 2, 2001):
        a = 1.7 * np.array([math.cos(gamma), math.sin(gamma)])
        # 2r - a a^T r / |a|^2  ==  Adasum(a, r) + Adasum(-a, r)
        y = oracle.adasum_pair(a, r) + oracle.adasum_pair(-a, r)
        np.testing.assert_allclose(y, 2 * r - a * (a @ r) / (a @ a), atol=1e-14)
        cos_eta = (r @ y) / np.linalg.norm(y)
        if cos_eta < worst:
            worst, worst_gamma = cos_eta, gamma
    assert abs(worst - golden["min_cos_eta"]) < 5e-5
    assert abs(worst - 2 * math.sqrt(2) / 3) < 1e-6
    assert abs(math.cos(worst_gamma) ** 2 - 2.0 / 3.0) < 2e-3
    assert abs(math.acos(worst) / math.pi - golden["max_angle_over_pi"]) < 5e-4


# -- Section 3.6: orthogonality measure is 1 (orthogonal) and 1/n (identical), n = 64 ----------
def test_nway_extremes_of_orthogonality_measure():
    golden = _golden("orthogonality_extremes.txt")
    n = int(golden["n_workers"])
    rng = _rng(7)
    width = 5
    ortho = [np.zeros(n * width) for _ in range(n)]
    for w in range(n):
        ortho[w][w * width:(w + 1) * width] = (1.0 + w) * rng.standard_normal(width)
    out, measure = oracle.adasum_reduce(ortho, return_orthogonality=True)
    np.testing.assert_allclose(out, np.sum(ortho, axis=0), rtol=0, atol=1e-14)
    assert abs(measure[0] - golden["orthogonal"]) < 1e-14
    g = rng.standard_normal(100)
    out, measure = oracle.adasum_reduce([g.copy() for _ in range(n)], return_orthogonality=True)
    np.testing.assert_allclose(out, g, rtol=1e-13)
    assert abs(measure[0] - golden["parallel_equal_norm"]) < 1e-14


# -- Section 3.4: recursive halves, written top-down in numpy, vs the bottom-up oracle ---------
def _pair_np(a, b):
    d, na, nb = a @ b, a @ a, b @ b
    ca = 1.0 if na == 0 else 1.0 - d / (2 * na)
    cb = 1.0 if nb == 0 else 1.0 - d / (2 * nb)
    return ca * a + cb * b


def _top_down(gs):
    if len(gs) == 1:
        return gs[0]
    half = len(gs) // 2
    return _pair_np(_top_down(gs[:half]), _top_down(gs[half:]))


@pytest.mark.parametrize("n", [2, 4, 8, 16])
def test_brute_force_top_down_tree(n):
    rng = _rng(100 + n)
    sizes = [1, 7, 64, 3, 33]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    shared = rng.standard_normal(offs[-1])
    gs = [0.6 * shared + rng.standard_normal(offs[-1]) * (0.1 + w) for w in range(n)]
    out = oracle.adasum_reduce(gs, offsets=offs)
    for t in range(len(sizes)):
        lo, hi = offs[t], offs[t + 1]
        ref = _top_down([g[lo:hi] for g in gs])
        np.testing.assert_allclose(out[lo:hi], ref, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("n", [3, 5, 6, 7, 11, 13, 24])
def test_top_down_order_for_any_count(n):
    """The top-down recursion of Section 3.4 for counts that are not powers of two: the oracle's
    `top_down` order against the same brute force; and it is a different tree from the bottom-up
    one with its carried operand (already for n = 3: bottom-up pairs (g0, g1) and carries g2,
    top-down pairs (g1, g2) first)."""
    rng = _rng(300 + n)
    sizes = [5, 40, 1]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    shared = rng.standard_normal(offs[-1])
    gs = [0.6 * shared + rng.standard_normal(offs[-1]) * (0.1 + w) for w in range(n)]
    out = oracle.adasum_reduce(gs, offsets=offs, top_down=True)
    for t in range(len(sizes)):
        lo, hi = offs[t], offs[t + 1]
        np.testing.assert_allclose(out[lo:hi], _top_down([g[lo:hi] for g in gs]), rtol=1e-12, atol=1e-14)
    bottom_up = oracle.adasum_reduce(gs, offsets=offs)
    assert np.linalg.norm(out - bottom_up) > 1e-3 * np.linalg.norm(bottom_up)


@pytest.mark.parametrize("n", [1, 2, 4, 8, 32])
def test_top_down_equals_bottom_up_for_powers_of_two(n):
    rng = _rng(400 + n)
    gs = [rng.standard_normal(50) for _ in range(n)]
    assert np.array_equal(oracle.adasum_reduce(gs, top_down=True), oracle.adasum_reduce(gs))


def test_tree_pairs_adjacent_workers_not_strided():
    """Level 1 pairs workers (0,1) and (2,3): with g0 = g1 and g2 = g3 orthogonal to g0 the
    result is g0 + g2; pairing (0,2),(1,3) would give (g0 + g2) as well only by accident of
    symmetry, so use unequal norms that separate the two trees."""
    rng = _rng(8)
    u, v = np.zeros(8), np.zeros(8)
    u[:4], v[4:] = rng.standard_normal(4), rng.standard_normal(4)
    gs = [u, 3 * u, v, v + u]
    adjacent = _pair_np(_pair_np(gs[0], gs[1]), _pair_np(gs[2], gs[3]))
    strided = _pair_np(_pair_np(gs[0], gs[2]), _pair_np(gs[1], gs[3]))
    assert _rel(adjacent, strided) > 1e-2
    np.testing.assert_allclose(oracle.adasum_reduce(gs), adjacent, rtol=1e-13)


def test_tree_and_linear_orders_differ_and_linear_matches_its_definition():
    rng = _rng(9)
    gs = [rng.standard_normal(50) + 0.3 for _ in range(4)]
    chain = gs[0]
    for g in gs[1:]:
        chain = _pair_np(chain, g)
    np.testing.assert_allclose(oracle.adasum_reduce(gs, linear_order=True), chain, rtol=1e-13)
    assert _rel(oracle.adasum_reduce(gs), chain) > 1e-3


def test_per_tensor_application_differs_from_whole_buffer():
    rng = _rng(10)
    a, b = rng.standard_normal(40), rng.standard_normal(40)
    b[:20] = a[:20]                              # first tensor identical, second independent
    per_tensor = oracle.adasum_pair(a, b, offsets=[0, 20, 40])
    np.testing.assert_allclose(per_tensor[:20], a[:20], rtol=1e-13)
    np.testing.assert_allclose(per_tensor[20:], _pair_np(a[20:], b[20:]), rtol=1e-13)
    assert _rel(per_tensor, oracle.adasum_pair(a, b)) > 1e-3


# -- zero-norm reading: a zero operand contributes nothing, the other passes through ----------
def test_zero_operands():
    b = _rng(11).standard_normal(31)
    z = np.zeros(31)
    np.testing.assert_array_equal(oracle.adasum_pair(z, b), b)
    np.testing.assert_array_equal(oracle.adasum_pair(b, z), b)
    np.testing.assert_array_equal(oracle.adasum_pair(z, z), z)
    gs = [z, b, z, z, 2 * b, z, z, z]            # zero leaves inside a deep tree
    out = oracle.adasum_reduce(gs)
    assert np.all(np.isfinite(out))
    np.testing.assert_allclose(out, 1.5 * b, rtol=1e-13)     # Adasum(b, 2b) = 3/2 b


# -- Appendix A.5 uses homogeneity: Adasum(s a, s b) = s Adasum(a, b) -------------------------
@pytest.mark.parametrize("s", [1e-6, -2.5, 1e5])
def test_homogeneity(s):
    rng = _rng(12)
    gs = [rng.standard_normal(77) + 0.2 for _ in range(8)]
    np.testing.assert_allclose(oracle.adasum_reduce([s * g for g in gs]),
                               s * oracle.adasum_reduce(gs), rtol=1e-12)


# -- Appendix A.3, Lemma (norm): each half operator has eigenvalues 1/2 and 1 -----------------
def test_norm_identity_and_bounds():
    rng = _rng(13)
    for trial in range(20):
        a, b = rng.standard_normal(19), rng.standard_normal(19) * rng.uniform(0.1, 10)
        d, na, nb = a @ b, a @ a, b @ b
        ca, cb = oracle.coefficients(d, na, nb)
        out = oracle.adasum_pair(a, b)
        assert abs(out @ out - (ca * ca * na + cb * cb * nb + 2 * ca * cb * d)) < 1e-11 * (na + nb)
        assert np.linalg.norm(out) <= math.sqrt(na) + math.sqrt(nb) + 1e-12
    gs = [rng.standard_normal(40) for _ in range(16)]
    assert np.linalg.norm(oracle.adasum_reduce(gs)) <= sum(np.linalg.norm(g) for g in gs)


# -- every tree node is a linear combination of the leaves: weights from the Gram matrix ------
@pytest.mark.parametrize("n", [2, 3, 5, 8, 16])
def test_gram_derived_leaf_weights_reproduce_the_tree(n):
    rng = _rng(200 + n)
    gs = np.stack([rng.standard_normal(48) + 0.4 for _ in range(n)])
    c = leaf_weights_from_gram(gs @ gs.T)
    np.testing.assert_allclose(oracle.adasum_reduce(list(gs)), c @ gs, rtol=1e-12, atol=1e-14)


# -- input conversion is exact for every stored format ----------------------------------------
def test_low_precision_inputs_are_converted_exactly():
    import torch

    vals = torch.tensor([0.0, -0.0, 1.0, -2.5, 6.0e-8, 6.1e-5, 65504.0, 1e-3, 0.333], dtype=torch.float32)
    for dt, name in ((torch.float16, "f16"), (torch.bfloat16, "bf16")):
        stored = vals.to(dt)
        exact = stored.to(torch.float64).numpy()
        bits = stored.view(torch.uint16).numpy() if name == "bf16" else stored.numpy()
        out = oracle.adasum_reduce([bits], dtype=name)          # N = 1 returns the input
        np.testing.assert_array_equal(out, exact)
        other = torch.flip(stored, dims=[0])
        obits = other.view(torch.uint16).numpy() if name == "bf16" else other.numpy()
        np.testing.assert_allclose(oracle.adasum_pair(bits, obits, dtype=name),
                                   _pair_np(exact, other.to(torch.float64).numpy()), rtol=1e-13)


def test_odd_worker_count_carries_the_last_operand():
    rng = _rng(14)
    gs = [rng.standard_normal(12) for _ in range(5)]
    ref = _pair_np(_pair_np(_pair_np(gs[0], gs[1]), _pair_np(gs[2], gs[3])), gs[4])
    np.testing.assert_allclose(oracle.adasum_reduce(gs), ref, rtol=1e-13)


def test_empty_tensors_are_allowed():
    rng = _rng(15)
    a, b = rng.standard_normal(10), rng.standard_normal(10)
    out = oracle.adasum_pair(a, b, offsets=[0, 0, 4, 4, 10])
    np.testing.assert_allclose(out[:4], _pair_np(a[:4], b[:4]), rtol=1e-13)
    np.testing.assert_allclose(out[4:], _pair_np(a[4:], b[4:]), rtol=1e-13)


def test_generator_statistics_level_one_coefficient():
    """Not a gate on the method: for the correlated-Gaussian generator with rho = 0.5 the
    level-one coefficients are close to 1 - rho/2 = 0.75."""
    from paper_2006_02924_b200 import workloads

    wl = workloads.generate("c1", tensor_sizes=[200_000])
    a, b = (g.double().numpy() for g in wl.grads)
    ca, cb = oracle.coefficients(float(a @ b), float(a @ a), float(b @ b))
    assert abs(ca - 0.75) < 0.01 and abs(cb - 0.75) < 0.01


# ---- the operator around a local optimizer step (Section 4.1) -------------------------------------

def _nearest_bf16_brute(x: float) -> int:
    """Nearest bf16 (ties to even) of a positive normal double, by trying both neighbours exactly."""
    from fractions import Fraction

    m, e = np.frexp(x)                          # x = m 2^e, 0.5 <= m < 1
    ulp = Fraction(2) ** (int(e) - 8)           # bf16 has 8 significant bits
    lo = int(Fraction(x) / ulp)                 # truncation, in units of ulp
    best = None
    for k in (lo, lo + 1):
        dist = abs(Fraction(x) - k * ulp)
        key = (dist, k & 1)                     # nearest, then even
        if best is None or key < best[0]:
            best = (key, k)
    value = float(best[1] * ulp)
    return int(np.array([value], dtype=np.float32).view(np.uint32)[0] >> 16)


def test_round_to_bf16_is_one_correct_rounding():
    rng = np.random.default_rng(77)
    xs = list(np.exp(rng.uniform(-20, 20, 400)))
    # traps for rounding in two steps: just above / below a bf16 midpoint, by less than an fp32 ulp
    xs += [1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 2.0 ** -8 - 2.0 ** -40, 1.0 + 3 * 2.0 ** -8 + 2.0 ** -45,
           1.0 + 3 * 2.0 ** -8 - 2.0 ** -45, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]
    got = oracle.round_to_dtype(np.array(xs), "bf16")
    want = [_nearest_bf16_brute(x) for x in xs]
    assert got.tolist() == want
    assert oracle.round_to_dtype(-np.array(xs), "bf16").tolist() == [w | 0x8000 for w in want]
    back = oracle.decode(got, "bf16")
    assert np.all(np.abs(back - np.array(xs)) <= np.array(xs) * 2.0 ** -8)


def test_delta_form_closed_cases():
    rng = np.random.default_rng(78)
    offsets = [0, 300, 300, 1000]
    start = rng.standard_normal(1000).astype(np.float32)
    # every worker took the same step, exactly representable: the result is that worker's state
    step = (rng.integers(-8, 9, 1000) * 2.0 ** -10).astype(np.float32)
    cur = (start.astype(np.float64) + step).astype(np.float32)
    exact = cur.astype(np.float64) - start == step
    out = oracle.adasum_reduce_delta([cur] * 4, start, offsets)
    assert np.allclose(out[exact], cur[exact].astype(np.float64), rtol=0, atol=1e-12)
    # steps with disjoint supports are orthogonal: the result is start plus all of them
    curs = []
    for w in range(4):
        d = np.zeros(1000, dtype=np.float32)
        d[w::4] = (rng.integers(1, 9, len(d[w::4])) * 2.0 ** -10).astype(np.float32)
        curs.append(((start.astype(np.float64) + d).astype(np.float32), d))
    out = oracle.adasum_reduce_delta([c for c, _ in curs], start, offsets)
    eff = sum((c.astype(np.float64) - start).astype(np.float32).astype(np.float64) for c, _ in curs)
    assert np.allclose(out, start + eff, rtol=0, atol=1e-12)
    # start = 0: the plain reduce
    g = [rng.standard_normal(1000).astype(np.float32) for _ in range(5)]
    assert np.array_equal(oracle.adasum_reduce_delta(g, np.zeros(1000, np.float32), offsets),
                          oracle.adasum_reduce(g, offsets))


def test_delta_form_rounds_the_difference_to_the_buffer_type():
    # 1 + 2^-11 is not an fp16; current - start must be what fp16 subtraction gives
    start = np.array([1.0, 1024.0, 0.5], dtype=np.float16)
    cur = np.array([1.001, 1025.0, 0.50049], dtype=np.float16)
    d = (cur.astype(np.float64) - start.astype(np.float64)).astype(np.float16)
    out = oracle.adasum_reduce_delta([cur, cur], start, dtype="f16")
    assert np.allclose(out, start.astype(np.float64) + d.astype(np.float64), rtol=0, atol=1e-15)


# ---- gradients stored with a scale (dynamic scaling, Section 4.4.1) ------------------------------

def test_scaled_form_orthogonal_workers_closed_case():
    """Orthogonal gradients add up.  The stored vectors are 4 x (1, 0) and 0.5 x (0, 1) with scales
    (4, 0.5): the result is (1, 1); multiplying by the scales instead of dividing gives (16, 0.25)."""
    a = np.array([4.0, 0.0])
    b = np.array([0.0, 0.5])
    got = oracle.adasum_reduce_scaled([a, b], [[4.0], [0.5]], dtype="f64")
    np.testing.assert_allclose(got, [1.0, 1.0], rtol=0, atol=1e-15)


def test_scaled_form_identical_gradients_whatever_the_scales():
    """Adasum(g, g, ..., g) = g: workers whose gradients are the same vector stored with different
    scales give that vector back, for every count and in every order."""
    rng = np.random.default_rng(5)
    g = rng.standard_normal(37)
    for n in (2, 3, 5, 8):
        scales = rng.uniform(0.01, 300.0, size=(n, 1))
        stored = [g * scales[w, 0] for w in range(n)]
        for kw in ({}, {"linear_order": True}, {"top_down": True}):
            got = oracle.adasum_reduce_scaled(stored, scales, dtype="f64", **kw)
            np.testing.assert_allclose(got, g, rtol=1e-13, atol=0)


def test_scaled_form_uniform_scale_is_homogeneity():
    """One scale s for every worker of a tensor: the operator is homogeneous of degree one, so the
    result is the plain reduce of the stored vectors divided by s, tensor by tensor."""
    rng = np.random.default_rng(6)
    offs = [0, 5, 5, 40, 41]
    n = 6
    stored = [rng.standard_normal(41) for _ in range(n)]
    per_tensor = np.array([3.0, 7.0, 0.125, 1000.0])
    scales = np.tile(per_tensor, (n, 1))
    got = oracle.adasum_reduce_scaled(stored, scales, offsets=offs, dtype="f64")
    plain = oracle.adasum_reduce(stored, offsets=offs, dtype="f64")
    for t in range(4):
        np.testing.assert_allclose(got[offs[t]:offs[t + 1]], plain[offs[t]:offs[t + 1]] / per_tensor[t],
                                   rtol=1e-13, atol=0)


def test_scaled_form_layout_is_worker_major_and_per_tensor():
    """Three workers, two tensors, six different power-of-two scales: the stored fp16 values are the
    gradients times their scale exactly, so the result must be the plain reduce of the gradients.
    Reading the table tensor-major, or applying a worker's scale to the wrong tensor, fails."""
    rng = np.random.default_rng(7)
    offs = [0, 9, 20]
    g = [np.round(rng.standard_normal(20) * 64) / 64 for _ in range(3)]        # exact in fp16 after scaling
    scales = np.array([[2.0, 0.25], [16.0, 0.5], [0.125, 8.0]])
    stored = []
    for w in range(3):
        v = g[w].copy()
        v[0:9] *= scales[w, 0]
        v[9:20] *= scales[w, 1]
        assert np.all(v.astype(np.float16).astype(np.float64) == v)
        stored.append(v.astype(np.float16))
    got = oracle.adasum_reduce_scaled(stored, scales, offsets=offs, dtype="f16")
    want = oracle.adasum_reduce(g, offsets=offs, dtype="f64")
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)


def test_scaled_form_orthogonality_is_that_of_the_gradients():
    """Mutually orthogonal gradients stored with different scales: the measure of Section 3.6 is 1."""
    n = 4
    stored = [np.eye(n)[w] * (w + 2.0) for w in range(n)]
    scales = np.array([[w + 2.0] for w in range(n)]) * 10.0
    out, ortho = oracle.adasum_reduce_scaled(stored, scales, dtype="f64", return_orthogonality=True)
    np.testing.assert_allclose(out, np.full(n, 0.1), rtol=1e-14)
    np.testing.assert_allclose(ortho, [1.0], rtol=1e-14)
