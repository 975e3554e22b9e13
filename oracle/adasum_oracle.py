"""Python face of the fp64 CPU oracle (``adasum_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The CUDA library and its Python binding never import this module, and this
module imports nothing from them.

The arithmetic lives in ``adasum_oracle.c`` (plain C, fp64, left-to-right sums); this file only
compiles it with gcc on first use and marshals numpy arrays.  Paper passages followed: the Adasum
pair operator (Section 3), its recursive binary-tree extension (Section 3.4, Algorithm 1's
bottom-up pairing), per-layer application (Sections 3.6 and 4.4.3), double accumulation and
gradients stored with a scale (Section 4.4.1) and the orthogonality measure (Section 3.6).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adasum_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libadasum_oracle.so")
_lock = threading.Lock()
_lib = None

_DTYPE_CODES = {"f32": 0, "f16": 1, "bf16": 2, "f64": 3}


def build(force: bool = False) -> str:
    """Compile the C oracle into ``oracle/_build`` (no-op when up to date)."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.adasum_oracle_reduce.restype = ctypes.c_int
            lib.adasum_oracle_reduce.argtypes = [
                ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.POINTER(ctypes.c_int64),
                ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                ctypes.POINTER(ctypes.c_double), ctypes.c_int,
            ]
            lib.adasum_oracle_coefficients.restype = None
            lib.adasum_oracle_coefficients.argtypes = [
                ctypes.c_double, ctypes.c_double, ctypes.c_double,
                ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
            ]
            lib.adasum_oracle_threads.restype = ctypes.c_int
            lib.adasum_oracle_threads.argtypes = [ctypes.c_int]
            _lib = lib
    return _lib


def _dtype_code(arr: np.ndarray, dtype: str | None) -> int:
    if dtype is None:
        dtype = {np.dtype(np.float32): "f32", np.dtype(np.float16): "f16",
                 np.dtype(np.float64): "f64"}.get(arr.dtype)
        if dtype is None:
            raise TypeError(f"pass dtype= for arrays of {arr.dtype} (bf16 travels as uint16)")
    if dtype == "bf16" and arr.dtype != np.uint16:
        raise TypeError("bf16 inputs are passed as their uint16 bit patterns")
    return _DTYPE_CODES[dtype]


def coefficients(dot: float, norm_a: float, norm_b: float) -> tuple[float, float]:
    """Scale factors of the pair operator from ``[a.b, a.a, b.b]`` (Algorithm 1)."""
    ca, cb = ctypes.c_double(), ctypes.c_double()
    _load().adasum_oracle_coefficients(dot, norm_a, norm_b, ctypes.byref(ca), ctypes.byref(cb))
    return ca.value, cb.value


def threads_used(threads: int = 0) -> int:
    return int(_load().adasum_oracle_threads(threads))


def adasum_reduce(grads, offsets=None, dtype: str | None = None, linear_order: bool = False,
                  return_orthogonality: bool = False, threads: int = 1, top_down: bool = False):
    """N-way Adasum of ``grads`` (a sequence of N equal-length 1-D arrays), per tensor.

    ``offsets`` (``num_tensors + 1`` element offsets) marks the tensors of the fused buffer;
    ``None`` means one tensor.  Returns the fp64 result (and, on request, the per-tensor
    orthogonality ``|Adasum(g_1..g_N)|^2 / sum_i |g_i|^2`` of Section 3.6).  ``linear_order``: the
    sequential recursion of Section 3.4; ``top_down``: its binary tree split by halves from the top
    (differs from the default bottom-up pairing only when N is not a power of two).
    """
    if linear_order and top_down:
        raise ValueError("choose one order")
    arrs = [np.ascontiguousarray(g).reshape(-1) for g in grads]
    n_workers = len(arrs)
    if n_workers < 1:
        raise ValueError("need at least one worker")
    total = arrs[0].size
    for a in arrs:
        if a.size != total or a.dtype != arrs[0].dtype:
            raise ValueError("all workers must have the same length and dtype")
    code = _dtype_code(arrs[0], dtype)
    if offsets is None:
        offsets = [0, total]
    offs = np.ascontiguousarray(np.asarray(offsets, dtype=np.int64))
    if offs[0] != 0 or offs[-1] != total or np.any(np.diff(offs) < 0):
        raise ValueError("offsets must start at 0, be non-decreasing and end at the buffer length")
    num_tensors = offs.size - 1
    out = np.zeros(total, dtype=np.float64)
    ortho = np.zeros(max(num_tensors, 1), dtype=np.float64)
    ptrs = (ctypes.c_void_p * n_workers)(*[a.ctypes.data for a in arrs])
    rc = _load().adasum_oracle_reduce(
        ptrs, code, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), num_tensors, n_workers,
        1 if linear_order else (2 if top_down else 0), out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
        ortho.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), threads)
    if rc != 0:
        raise MemoryError("adasum_oracle_reduce failed")
    if return_orthogonality:
        return out, ortho[:num_tensors]
    return out


def adasum_pair(a, b, offsets=None, dtype: str | None = None) -> np.ndarray:
    """One application of the operator, per tensor: ``Adasum(a, b)``."""
    return adasum_reduce([a, b], offsets=offsets, dtype=dtype)


# ---- the operator wrapped around a local optimizer step -----------------------------------------

def decode(arr: np.ndarray, dtype: str | None = None) -> np.ndarray:
    """The stored values as fp64, exactly (bf16 travels as uint16 bit patterns)."""
    arr = np.asarray(arr)
    if dtype == "bf16":
        if arr.dtype != np.uint16:
            raise TypeError("bf16 inputs are passed as their uint16 bit patterns")
        return (arr.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return arr.astype(np.float64)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """fp64 values rounded ONCE, to nearest even, to f32 / f16 / bf16 (bf16 as uint16 patterns);
    f64 is returned as it is."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f64":
        return x
    if dtype == "f32":
        return x.astype(np.float32)
    if dtype == "f16":
        return x.astype(np.float16)
    if dtype != "bf16":
        raise ValueError(dtype)
    # fp64 -> fp32 with round-to-odd (truncate, then set the last bit if anything was lost), so
    # that the second rounding, fp32 -> bf16 to nearest even, sees whether the value was above or
    # below a midpoint: together one correct rounding.
    f = x.astype(np.float32)
    inexact = f.astype(np.float64) != x
    too_big = np.abs(f.astype(np.float64)) > np.abs(x)
    f = np.where(too_big, np.nextafter(f, np.float32(0)), f).astype(np.float32)
    bits = f.view(np.uint32) | inexact.astype(np.uint32)
    rounded = (bits.astype(np.uint64) + 0x7FFF + ((bits >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def adasum_reduce_delta(currents, start, offsets=None, dtype: str | None = None, linear_order: bool = False,
                        return_orthogonality: bool = False, threads: int = 1):
    """``start + Adasum_w(currents[w] - start)`` per tensor (Section 4.1: the operator is applied to
    the effective gradients of a local optimizer step and the combination is added back to the
    parameters the step started from).  Each difference is rounded once to the buffers' own type,
    as ``current - start`` is in a framework; everything after that is fp64.  Returns fp64."""
    if dtype is None:
        dtype = {np.dtype(np.float32): "f32", np.dtype(np.float16): "f16",
                 np.dtype(np.float64): "f64"}[np.asarray(start).dtype]
    s = decode(start, dtype)
    deltas = [round_to_dtype(decode(c, dtype) - s, dtype) for c in currents]
    res = adasum_reduce(deltas, offsets=offsets, dtype=dtype, linear_order=linear_order,
                        return_orthogonality=return_orthogonality, threads=threads)
    if return_orthogonality:
        return s + res[0], res[1]
    return s + res


# ---- gradients stored with a scale -------------------------------------------------------------

def adasum_reduce_scaled(grads, scales, offsets=None, dtype: str | None = None, linear_order: bool = False,
                         return_orthogonality: bool = False, threads: int = 1, top_down: bool = False):
    """Dynamic scaling (Section 4.4.1): worker w's buffer holds ``scales[w][t]`` times its gradient
    for tensor t.  By definition the result is the operator applied to the gradients themselves:
    every stored value is decoded to fp64 and divided by its scale, then ``adasum_reduce`` runs on
    those fp64 vectors.  Returns fp64."""
    arrs = [decode(g, dtype).reshape(-1) for g in grads]
    total = arrs[0].size
    offs = np.asarray([0, total] if offsets is None else offsets, dtype=np.int64)
    num_tensors = offs.size - 1
    sc = np.asarray(scales, dtype=np.float64).reshape(len(arrs), num_tensors)
    true = []
    for w, a in enumerate(arrs):
        g = a.copy()
        for t in range(num_tensors):
            g[offs[t]:offs[t + 1]] /= sc[w, t]
        true.append(g)
    return adasum_reduce(true, offsets=offs, dtype="f64", linear_order=linear_order,
                         return_orthogonality=return_orthogonality, threads=threads, top_down=top_down)
