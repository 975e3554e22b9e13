"""Thin ctypes binding of the C ABI in ``include/adasum.h``: argument marshalling only.

Every function has the name of the C entry point it calls.  PyTorch is used for device memory
and streams; all arithmetic runs in the CUDA library.  There is no CPU fallback: importing this
module raises if the native library has not been built.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "lib", "libadasum_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"native library {LIB_PATH} is missing; build it with "
        "`python -m paper_2006_02924_b200.build` (needs nvcc, targets sm_100a)")

_lib = ctypes.CDLL(LIB_PATH)

ADASUM_F32, ADASUM_F16, ADASUM_BF16, ADASUM_F64 = 0, 1, 2, 3
ADASUM_FLAG_SIMPLE_KERNELS, ADASUM_FLAG_SEPARATE_FINISH, ADASUM_FLAG_LINEAR_ORDER = 1 << 16, 1 << 17, 1 << 18
ADASUM_FLAG_NO_TCGEN05 = 1 << 19
ADASUM_FLAG_TOP_DOWN_HALVES = 1 << 20
ADASUM_FLAG_NO_LEVEL_FUSION = 1 << 21
ADASUM_FLAG_SELFTEST_TIMEOUT = 1 << 22
ADASUM_OK = 0
ADASUM_MAX_WORKERS = 4096
ADASUM_MAX_LEVELS = 12
_DTYPES = {torch.float32: ADASUM_F32, torch.float16: ADASUM_F16, torch.bfloat16: ADASUM_BF16,
           torch.float64: ADASUM_F64}

_i64p = ctypes.POINTER(ctypes.c_int64)
_i32p = ctypes.POINTER(ctypes.c_int32)

_lib.adasum_workspace_bytes.restype = ctypes.c_size_t
_lib.adasum_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int,
                                        ctypes.c_uint32]
_lib.adasum_plan_info.restype = ctypes.c_int
_lib.adasum_plan_info.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int,
                                  ctypes.c_uint32, _i32p, _i32p, _i32p]
_lib.adasum_reduce.restype = ctypes.c_int
_lib.adasum_reduce.argtypes = [ctypes.POINTER(ctypes.c_void_p), _i64p, ctypes.c_int32, ctypes.c_int32,
                               ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                               ctypes.c_uint32, ctypes.c_void_p]
_lib.adasum_reduce_ex.restype = ctypes.c_int
_lib.adasum_reduce_ex.argtypes = [ctypes.POINTER(ctypes.c_void_p), _i64p, ctypes.c_int32, ctypes.c_int32,
                                  ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                  ctypes.c_uint32, ctypes.c_void_p]
_lib.adasum_reduce_delta.restype = ctypes.c_int
_lib.adasum_reduce_delta.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, _i64p, ctypes.c_int32,
                                     ctypes.c_int32, ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32, ctypes.c_void_p]
_lib.adasum_pair.restype = ctypes.c_int
_lib.adasum_pair.argtypes = [ctypes.c_void_p, ctypes.c_void_p, _i64p, ctypes.c_int32, ctypes.c_int,
                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32,
                             ctypes.c_void_p]
_lib.adasum_status_string.restype = ctypes.c_char_p
_lib.adasum_status_string.argtypes = [ctypes.c_int]
_lib.adasum_last_error.restype = ctypes.c_char_p
_lib.adasum_last_error.argtypes = []
_lib.adasum_shutdown.restype = ctypes.c_int
_lib.adasum_shutdown.argtypes = []


class AdasumError(RuntimeError):
    def __init__(self, status: int):
        self.status = int(status)
        detail = _lib.adasum_last_error().decode()
        super().__init__(f"{adasum_status_string(status)}: {detail}" if detail else adasum_status_string(status))


def flags_radix(first: int = 0, later: int = 0) -> int:
    """Value of the ``flags`` argument that fixes the radix of the first / later levels."""
    return (first & 0xFF) | ((later & 0xFF) << 8)


def adasum_status_string(status: int) -> str:
    return _lib.adasum_status_string(int(status)).decode()


def adasum_last_error() -> str:
    return _lib.adasum_last_error().decode()


def adasum_shutdown() -> None:
    status = _lib.adasum_shutdown()
    if status != ADASUM_OK:
        raise AdasumError(status)


def adasum_workspace_bytes(total_elems: int, num_tensors: int, n_workers: int, dtype, flags: int = 0) -> int:
    return int(_lib.adasum_workspace_bytes(int(total_elems), int(num_tensors), int(n_workers),
                                           _dtype_code(dtype), int(flags)))


def adasum_plan_info(total_elems: int, num_tensors: int, n_workers: int, dtype, flags: int = 0) -> dict:
    radices = (ctypes.c_int32 * ADASUM_MAX_LEVELS)()
    levels, launches = ctypes.c_int32(), ctypes.c_int32()
    status = _lib.adasum_plan_info(int(total_elems), int(num_tensors), int(n_workers), _dtype_code(dtype),
                                   int(flags), radices, ctypes.byref(levels), ctypes.byref(launches))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return {"radices": [int(radices[i]) for i in range(levels.value)], "launches": int(launches.value)}


_lib.adasum_device_status.restype = ctypes.c_int
_lib.adasum_device_status.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int, ctypes.c_uint32,
                                      ctypes.c_void_p, ctypes.c_void_p]


def adasum_device_status(total_elems: int, num_tensors: int, n_workers: int, dtype, workspace, flags: int = 0,
                         stream=None) -> int:
    """``adasum_device_status`` of the C ABI: 0, or 7 (ADASUM_ERR_TIMEOUT) if a bounded device-side
    wait of the last reduce on ``workspace`` ran out.  Synchronises the stream."""
    return int(_lib.adasum_device_status(int(total_elems), int(num_tensors), int(n_workers), _dtype_code(dtype),
                                         int(flags), workspace.data_ptr(), _stream_handle(stream)))


def _dtype_code(dtype) -> int:
    if isinstance(dtype, int):
        return dtype
    if isinstance(dtype, str):
        return {"f32": ADASUM_F32, "f16": ADASUM_F16, "bf16": ADASUM_BF16, "f64": ADASUM_F64}[dtype]
    return _DTYPES[dtype]


def _offsets_array(offsets, total: int) -> np.ndarray:
    if offsets is None:
        offsets = [0, total]
    return np.ascontiguousarray(np.asarray(offsets, dtype=np.int64))


def _stream_handle(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _workspace(workspace, need: int, device):
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
    return workspace, workspace.data_ptr(), workspace.numel() * workspace.element_size()


def adasum_reduce(grads, tensor_offsets=None, out=None, workspace=None, flags: int = 0, stream=None):
    """``adasum_reduce`` of the C ABI.  ``grads``: N CUDA tensors (one fused buffer per worker, same
    dtype and length).  Returns ``out`` (fp32, allocated here if not given)."""
    grads = list(grads)
    first = grads[0]
    total = first.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=first.device)
    need = adasum_workspace_bytes(total, num_tensors, len(grads), first.dtype, flags)
    workspace, ws_ptr, ws_bytes = _workspace(workspace, need, first.device)
    ptrs = (ctypes.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    with torch.cuda.device(first.device):
        status = _lib.adasum_reduce(ptrs, offs.ctypes.data_as(_i64p), num_tensors, len(grads),
                                    _dtype_code(first.dtype), out.data_ptr(), ws_ptr, ws_bytes, int(flags),
                                    _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out


def adasum_reduce_ex(grads, tensor_offsets=None, out=None, orthogonality=None, workspace=None, flags: int = 0,
                     stream=None):
    """``adasum_reduce_ex`` of the C ABI: the reduce plus the per-tensor orthogonality measure.
    Returns ``(out, orthogonality)`` (both allocated here if not given)."""
    grads = list(grads)
    first = grads[0]
    total = first.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=first.device)
    if orthogonality is None:
        orthogonality = torch.empty(max(num_tensors, 1), dtype=torch.float32, device=first.device)[:num_tensors]
    need = adasum_workspace_bytes(total, num_tensors, len(grads), first.dtype, flags)
    workspace, ws_ptr, ws_bytes = _workspace(workspace, need, first.device)
    ptrs = (ctypes.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    with torch.cuda.device(first.device):
        status = _lib.adasum_reduce_ex(ptrs, offs.ctypes.data_as(_i64p), num_tensors, len(grads),
                                       _dtype_code(first.dtype), out.data_ptr(), orthogonality.data_ptr(), ws_ptr,
                                       ws_bytes, int(flags), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out, orthogonality


_lib.adasum_reduce_scaled.restype = ctypes.c_int
_lib.adasum_reduce_scaled.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, _i64p, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32, ctypes.c_void_p]


def adasum_reduce_scaled(grads, scales, tensor_offsets=None, out=None, orthogonality=None, workspace=None,
                         flags: int = 0, stream=None, want_orthogonality: bool = False):
    """``adasum_reduce_scaled`` of the C ABI: the buffers hold ``scales[w, t]`` times worker w's
    gradient for tensor t (a CUDA fp32 tensor of shape [N, num_tensors]); returns the combination of
    the gradients themselves (and the orthogonality measure when asked for)."""
    grads = list(grads)
    first = grads[0]
    total = first.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if scales.dtype != torch.float32 or not scales.is_cuda or not scales.is_contiguous():
        raise TypeError("scales must be a contiguous CUDA fp32 tensor")
    if scales.numel() != len(grads) * num_tensors:
        raise ValueError(f"scales has {scales.numel()} entries, need {len(grads)} x {num_tensors}")
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=first.device)
    if orthogonality is None and want_orthogonality:
        orthogonality = torch.empty(max(num_tensors, 1), dtype=torch.float32, device=first.device)[:num_tensors]
    need = adasum_workspace_bytes(total, num_tensors, len(grads), first.dtype, flags)
    workspace, ws_ptr, ws_bytes = _workspace(workspace, need, first.device)
    ptrs = (ctypes.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    with torch.cuda.device(first.device):
        status = _lib.adasum_reduce_scaled(ptrs, scales.data_ptr(), offs.ctypes.data_as(_i64p), num_tensors,
                                           len(grads), _dtype_code(first.dtype), out.data_ptr(),
                                           orthogonality.data_ptr() if orthogonality is not None else None, ws_ptr,
                                           ws_bytes, int(flags), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return (out, orthogonality) if orthogonality is not None else out


_lib.adasum_sharded_gram.restype = ctypes.c_int
_lib.adasum_sharded_gram.argtypes = [ctypes.POINTER(ctypes.c_void_p), _i64p, ctypes.c_int32, ctypes.c_int32,
                                     ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32, ctypes.c_int32,
                                     ctypes.POINTER(ctypes.c_size_t), _i64p, ctypes.c_void_p]
_lib.adasum_sharded_apply.restype = ctypes.c_int
_lib.adasum_sharded_apply.argtypes = [ctypes.POINTER(ctypes.c_void_p), _i64p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_size_t, ctypes.c_uint32, ctypes.c_int32, ctypes.c_void_p]


def adasum_reduce_delta(currents, start, tensor_offsets=None, out=None, out_dtype=None, orthogonality=None,
                        workspace=None, flags: int = 0, stream=None):
    """``adasum_reduce_delta`` of the C ABI: ``out = start + Adasum_w(currents[w] - start)`` per
    tensor.  ``start=None`` gives the plain reduce with a choice of output type.  ``out`` may be
    ``start`` itself (in-place update) when the types agree.  Returns ``out``."""
    currents = list(currents)
    first = currents[0]
    total = first.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if out is None:
        out = torch.empty(total, dtype=out_dtype or torch.float32, device=first.device)
    need = adasum_workspace_bytes(total, num_tensors, len(currents), first.dtype, flags)
    workspace, ws_ptr, ws_bytes = _workspace(workspace, need, first.device)
    ptrs = (ctypes.c_void_p * len(currents))(*[g.data_ptr() for g in currents])
    if start is not None and (start.dtype != first.dtype or start.numel() != total):
        raise ValueError("start must have the type and size of the workers' buffers")
    with torch.cuda.device(first.device):
        status = _lib.adasum_reduce_delta(ptrs, None if start is None else start.data_ptr(),
                                          offs.ctypes.data_as(_i64p), num_tensors, len(currents),
                                          _dtype_code(first.dtype), out.data_ptr(), _dtype_code(out.dtype),
                                          None if orthogonality is None else orthogonality.data_ptr(),
                                          ws_ptr, ws_bytes, int(flags), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out


def adasum_sharded_gram(grads, tensor_offsets, workspace, level: int, flags: int = 0, stream=None):
    """``adasum_sharded_gram`` of the C ABI.  Returns this GPU's fp64 Gram sums of ``level`` as a
    float64 view INTO ``workspace`` (add it over the GPUs in place, then call ``adasum_sharded_apply``)."""
    grads = list(grads)
    first = grads[0]
    offs = _offsets_array(tensor_offsets, first.numel())
    ptrs = (ctypes.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    off, count = ctypes.c_size_t(), ctypes.c_int64()
    with torch.cuda.device(first.device):
        status = _lib.adasum_sharded_gram(ptrs, offs.ctypes.data_as(_i64p), offs.size - 1, len(grads),
                                          _dtype_code(first.dtype), workspace.data_ptr(),
                                          workspace.numel() * workspace.element_size(), int(flags), int(level),
                                          ctypes.byref(off), ctypes.byref(count), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return workspace.view(torch.uint8)[off.value:off.value + 8 * count.value].view(torch.float64)


def adasum_sharded_apply(grads, tensor_offsets, out, workspace, level: int, orthogonality=None, flags: int = 0,
                         stream=None):
    """``adasum_sharded_apply`` of the C ABI."""
    grads = list(grads)
    first = grads[0]
    offs = _offsets_array(tensor_offsets, first.numel())
    ptrs = (ctypes.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    with torch.cuda.device(first.device):
        status = _lib.adasum_sharded_apply(ptrs, offs.ctypes.data_as(_i64p), offs.size - 1, len(grads),
                                           _dtype_code(first.dtype), out.data_ptr(),
                                           None if orthogonality is None else orthogonality.data_ptr(),
                                           workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                           int(flags), int(level), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out


def adasum_reduce_sharded(grads, tensor_offsets, group=None, out=None, orthogonality=None, workspace=None,
                          flags: int = 0, stream=None):
    """The whole element-sharded reduce on this rank: per level ``adasum_sharded_gram``, a
    ``torch.distributed.all_reduce`` (sum) of the Gram sums over ``group``, ``adasum_sharded_apply``.
    ``grads`` are this rank's slices (see ``include/adasum.h``).  Returns this rank's slice of the result."""
    import torch.distributed as dist

    grads = list(grads)
    first = grads[0]
    total = first.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=first.device)
    need = adasum_workspace_bytes(total, num_tensors, len(grads), first.dtype, flags)
    workspace, _, _ = _workspace(workspace, need, first.device)
    levels = len(adasum_plan_info(total, num_tensors, len(grads), first.dtype, flags)["radices"])
    for level in range(levels):
        sums = adasum_sharded_gram(grads, offs, workspace, level, flags=flags, stream=stream)
        if sums.numel() > 0:
            dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
        adasum_sharded_apply(grads, offs, out, workspace, level, orthogonality=orthogonality, flags=flags,
                             stream=stream)
    return out


def adasum_pair(a, b, tensor_offsets=None, out=None, workspace=None, flags: int = 0, stream=None):
    """``adasum_pair`` of the C ABI: ``out = Adasum(a, b)`` per tensor."""
    total = a.numel()
    offs = _offsets_array(tensor_offsets, total)
    num_tensors = offs.size - 1
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=a.device)
    need = adasum_workspace_bytes(total, num_tensors, 2, a.dtype, flags)
    workspace, ws_ptr, ws_bytes = _workspace(workspace, need, a.device)
    with torch.cuda.device(a.device):
        status = _lib.adasum_pair(a.data_ptr(), b.data_ptr(), offs.ctypes.data_as(_i64p), num_tensors,
                                  _dtype_code(a.dtype), out.data_ptr(), ws_ptr, ws_bytes, int(flags),
                                  _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out


def raw():
    """The loaded ``ctypes.CDLL`` (for tests that pass raw pointers)."""
    return _lib


class _LaunchRecord(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("level", ctypes.c_int32), ("radix", ctypes.c_int32),
                ("ms", ctypes.c_float)]


KERNEL_NAMES = {0: "gram_partial", 1: "tree_weights", 2: "weighted_sum", 3: "convert", 4: "fused_small",
                5: "wsum_gram", 6: "short_tensors"}

_lib.adasum_profile_enable.restype = ctypes.c_int
_lib.adasum_profile_enable.argtypes = [ctypes.c_int32]
_lib.adasum_profile_collect.restype = ctypes.c_int
_lib.adasum_profile_collect.argtypes = [ctypes.POINTER(_LaunchRecord), ctypes.c_int32, _i32p]


def adasum_profile_enable(max_launches: int) -> None:
    status = _lib.adasum_profile_enable(int(max_launches))
    if status != ADASUM_OK:
        raise AdasumError(status)


def adasum_profile_collect(capacity: int = 4096) -> list[dict]:
    """One dict per kernel launch since ``adasum_profile_enable``: kernel, level, radix, ms."""
    records = (_LaunchRecord * capacity)()
    count = ctypes.c_int32()
    status = _lib.adasum_profile_collect(records, capacity, ctypes.byref(count))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return [{"kernel": KERNEL_NAMES.get(r.kernel, str(r.kernel)), "level": r.level, "radix": r.radix,
             "ms": float(r.ms)} for r in records[:min(count.value, capacity)]]


ADASUM_NOALLOC_MAX_ELEMS = 1 << 26
ADASUM_NOALLOC_MAX_TENSORS = 4096

_lib.adasum_pair_noalloc.restype = ctypes.c_int
_lib.adasum_pair_noalloc.argtypes = [ctypes.c_void_p, ctypes.c_void_p, _i64p, ctypes.c_int32, ctypes.c_int,
                                     ctypes.c_void_p, ctypes.c_void_p]


def adasum_pair_noalloc(a, b, tensor_offsets=None, out=None, stream=None):
    """``adasum_pair_noalloc`` of the C ABI: the pair operator for callers that cannot allocate
    device memory.  The library uses a fixed scratch array of its own instead of a workspace, so
    pass ``out`` to keep this wrapper from allocating either (it allocates ``out`` with torch only
    when none is given)."""
    total = a.numel()
    offs = _offsets_array(tensor_offsets, total)
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=a.device)
    with torch.cuda.device(a.device):
        status = _lib.adasum_pair_noalloc(a.data_ptr(), b.data_ptr(), offs.ctypes.data_as(_i64p), offs.size - 1,
                                          _dtype_code(a.dtype), out.data_ptr(), _stream_handle(stream))
    if status != ADASUM_OK:
        raise AdasumError(status)
    return out
