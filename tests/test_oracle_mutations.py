"""Do the oracle's pins have teeth?  Plausible mistakes are planted in COPIES of the oracle's C
source (a dropped factor, a transposed norm, a wrong sign, strided instead of adjacent pairing, a
missing zero rule, whole-buffer instead of per-tensor dots); each copy is compiled on the CPU and
must fail at least one of the checks that the paper and the mathematics fix.  The unmodified
source must pass them all."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "adasum_oracle.c")


def _compile(source_text, tmp_path, name):
    c_path = tmp_path / f"{name}.c"
    so_path = tmp_path / f"lib{name}.so"
    c_path.write_text(source_text)
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-o", str(so_path), str(c_path), "-lm"])
    lib = ctypes.CDLL(str(so_path))
    lib.adasum_oracle_reduce.restype = ctypes.c_int
    lib.adasum_oracle_reduce.argtypes = [
        ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_int,
        ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), ctypes.c_int]

    def reduce(grads, offsets=None):
        arrs = [np.ascontiguousarray(g, dtype=np.float64) for g in grads]
        total = arrs[0].size
        offs = np.ascontiguousarray(np.asarray([0, total] if offsets is None else offsets, dtype=np.int64))
        out = np.zeros(total)
        ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
        rc = lib.adasum_oracle_reduce(ptrs, 3, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), offs.size - 1,
                                      len(arrs), 0, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), None, 1)
        assert rc == 0
        return out

    return reduce


def _pair(a, b):
    d, na, nb = a @ b, a @ a, b @ b
    ca = 1.0 if na == 0 else 1.0 - d / (2 * na)
    cb = 1.0 if nb == 0 else 1.0 - d / (2 * nb)
    return ca * a + cb * b


def _failed_pins(reduce):
    """Names of the pins that `reduce` violates."""
    rng = np.random.default_rng(42)
    failed = []

    def check(name, got, want, tol=1e-12):
        if not (np.all(np.isfinite(got)) and np.linalg.norm(got - want) <= tol * max(np.linalg.norm(want), 1e-300)):
            failed.append(name)

    a, b = np.zeros(16), np.zeros(16)
    a[0::2], b[1::2] = rng.standard_normal(8), 3 * rng.standard_normal(8)
    check("orthogonal pair is the plain sum", reduce([a, b]), a + b)
    g = rng.standard_normal(33)
    for c in (1.0, 2.0, -3.0):
        check(f"Adasum(g, {c} g) = (1 + c)/2 g", reduce([g, c * g]), 0.5 * (1 + c) * g)
    x, y = rng.standard_normal(20), 0.3 * rng.standard_normal(20) + 0.2
    check("mean of the two visiting orders", reduce([x, y]),
          0.5 * ((x + (1 - (x @ y) / (y @ y)) * y) + (y + (1 - (x @ y) / (x @ x)) * x)))
    check("symmetric in its arguments", reduce([x, y]), reduce([y, x]))
    z = np.zeros(20)
    check("zero operand passes the other through", reduce([z, x]), x)
    check("zero operand passes the other through (right)", reduce([x, z]), x)
    u, v = np.zeros(8), np.zeros(8)
    u[:4], v[4:] = rng.standard_normal(4), rng.standard_normal(4)
    gs = [u, 3 * u, v, v + u]
    check("level one pairs workers (0,1) and (2,3)", reduce(gs), _pair(_pair(gs[0], gs[1]), _pair(gs[2], gs[3])))
    hs = [rng.standard_normal(12) + 0.3 for _ in range(8)]

    def top_down(v):
        return v[0] if len(v) == 1 else _pair(top_down(v[:len(v) // 2]), top_down(v[len(v) // 2:]))

    check("recursive halves (top-down brute force)", reduce(hs), top_down(hs))
    p, q = rng.standard_normal(40), rng.standard_normal(40)
    q[:20] = p[:20]
    want = np.concatenate([p[:20], _pair(p[20:], q[20:])])
    check("dots are per tensor, not per buffer", reduce([p, q], offsets=[0, 20, 40]), want)
    five = [rng.standard_normal(9) for _ in range(5)]
    check("odd count carries the last operand", reduce(five),
          _pair(_pair(_pair(five[0], five[1]), _pair(five[2], five[3])), five[4]))
    return failed


MUTATIONS = {
    "dropped factor two": ("1.0 - dot / (2.0 * norm_a)", "1.0 - dot / (norm_a)"),
    "transposed norms": ("*coef_b = (norm_b == 0.0) ? 1.0 : 1.0 - dot / (2.0 * norm_b);",
                         "*coef_b = (norm_b == 0.0) ? 1.0 : 1.0 - dot / (2.0 * norm_a);"),
    "wrong sign": ("*coef_a = (norm_a == 0.0) ? 1.0 : 1.0 - dot", "*coef_a = (norm_a == 0.0) ? 1.0 : 1.0 + dot"),
    "norm instead of squared norm": ("norm_a += a[e] * a[e];", "norm_a += fabs(a[e]);"),
    "no zero rule": ("*coef_a = (norm_a == 0.0) ? 1.0 : ", "*coef_a = "),
    # workers paired at distance n/2 instead of as neighbours (done where the leaves are loaded, so
    # that the mutant stays memory-safe)
    "strided pairing": ("x[w][e] = element_as_double(grads[w], dtype, begin + e);",
                        "x[w][e] = element_as_double(grads[(w % 2) * (n_workers / 2) + w / 2], dtype, begin + e);"),
    "dot over the whole buffer": ("x[w][e] = element_as_double(grads[w], dtype, begin + e);",
                                  "x[w][e] = element_as_double(grads[w], dtype, e);"),
    "carry dropped": ("        m = (m + 1) / 2;", "        m = m / 2;"),
    "coefficient applied to the wrong operand": ("dst[e] = ca * a[e] + cb * b[e];", "dst[e] = cb * a[e] + ca * b[e];"),
}


def test_unmodified_oracle_passes_every_pin(tmp_path):
    assert _failed_pins(_compile(open(SRC).read(), tmp_path, "original")) == []


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(tmp_path, name):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for '{name}' not found in the oracle source"
    mutant = _compile(text.replace(old, new, 1), tmp_path, "mutant")
    assert _failed_pins(mutant), f"no pin notices: {name}"


# ---- the scaled form (its oracle function is Python around the same C tree) -----------------------

def _scaled_variant(mistake):
    """oracle.adasum_reduce_scaled with one plausible mistake planted (None: as it stands)."""
    from oracle import adasum_oracle as oracle

    def scaled(grads, scales, offsets=None, dtype=None, **kw):
        arrs = [oracle.decode(g, dtype).reshape(-1) for g in grads]
        total = arrs[0].size
        offs = np.asarray([0, total] if offsets is None else offsets, dtype=np.int64)
        num_tensors = offs.size - 1
        sc = np.asarray(scales, dtype=np.float64)
        if mistake == "table read tensor-major":
            sc = sc.reshape(-1).reshape(num_tensors, len(arrs)).T
        else:
            sc = sc.reshape(len(arrs), num_tensors)
        true = []
        for w, a in enumerate(arrs):
            g = a.copy()
            for t in range(num_tensors):
                s = sc[w, 0] if mistake == "first tensor's scale for every tensor" else sc[w, t]
                if mistake == "multiplied instead of divided":
                    g[offs[t]:offs[t + 1]] *= s
                elif mistake == "worker 0's scale for every worker":
                    g[offs[t]:offs[t + 1]] /= sc[0, t]
                else:
                    g[offs[t]:offs[t + 1]] /= s
            true.append(g)
        if mistake == "scales undone on the output instead":
            plain = oracle.adasum_reduce(arrs, offsets=offs, dtype="f64", **kw)
            res = plain[0] if isinstance(plain, tuple) else plain
            for t in range(num_tensors):
                res[offs[t]:offs[t + 1]] /= sc[:, t].mean()
            return plain
        return oracle.adasum_reduce(true, offsets=offs, dtype="f64", **kw)

    return scaled


def _failed_scaled_pins(scaled):
    from oracle import adasum_oracle as oracle

    failed = []

    def check(name, got, want, tol=1e-12):
        if not (np.all(np.isfinite(got)) and np.linalg.norm(got - want) <= tol * max(np.linalg.norm(want), 1e-300)):
            failed.append(name)

    check("orthogonal workers add up", scaled([np.array([4.0, 0.0]), np.array([0.0, 0.5])], [[4.0], [0.5]], dtype="f64"),
          np.array([1.0, 1.0]))
    rng = np.random.default_rng(5)
    g = rng.standard_normal(37)
    sc = rng.uniform(0.01, 300.0, size=(5, 1))
    check("identical gradients under any scales", scaled([g * sc[w, 0] for w in range(5)], sc, dtype="f64"), g)
    offs = [0, 9, 20]
    gs = [np.round(rng.standard_normal(20) * 64) / 64 for _ in range(3)]
    table = np.array([[2.0, 0.25], [16.0, 0.5], [0.125, 8.0]])
    stored = []
    for w in range(3):
        v = gs[w].copy()
        v[0:9] *= table[w, 0]
        v[9:20] *= table[w, 1]
        stored.append(v.astype(np.float16))
    check("six power-of-two scales, fp16 storage", scaled(stored, table, offsets=offs, dtype="f16"),
          oracle.adasum_reduce(gs, offsets=offs, dtype="f64"))
    return failed


SCALED_MISTAKES = ["multiplied instead of divided", "table read tensor-major", "first tensor's scale for every tensor",
                   "worker 0's scale for every worker", "scales undone on the output instead"]


def test_scaled_form_as_it_stands_passes_its_pins():
    from oracle import adasum_oracle as oracle

    assert _failed_scaled_pins(oracle.adasum_reduce_scaled) == []
    assert _failed_scaled_pins(_scaled_variant(None)) == []


@pytest.mark.parametrize("mistake", SCALED_MISTAKES)
def test_planted_mistake_in_the_scaled_form_is_caught(mistake):
    assert _failed_scaled_pins(_scaled_variant(mistake)), mistake
