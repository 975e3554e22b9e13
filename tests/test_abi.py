"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes its workspace sensibly and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2006_02924_b200 import build

    build.build()
    from paper_2006_02924_b200 import binding as b

    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "adasum.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adasum_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(binding):
    names = _declared_functions()
    assert {"adasum_reduce", "adasum_pair", "adasum_workspace_bytes", "adasum_status_string"} <= set(names)
    lib = binding.raw()
    for name in names:
        assert hasattr(lib, name), f"{name} declared in adasum.h but not exported"


def test_binding_exposes_the_same_names(binding):
    for name in _declared_functions():
        assert hasattr(binding, name), name


def test_status_strings(binding):
    seen = {binding.adasum_status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ADASUM_OK" in seen and "ADASUM_ERR_WORKSPACE" in seen
    assert binding.adasum_status_string(99) == "ADASUM_ERR_UNKNOWN"


def test_workspace_bytes(binding):
    ws = binding.adasum_workspace_bytes
    assert ws(0, 0, 1, "f32") > 0
    assert ws(-1, 1, 2, "f32") == 0
    assert ws(10, 1, 0, "f32") == 0
    assert ws(10, 1, 2, 7) == 0
    assert ws(10, 1, 2, "f32", 3) == 0                       # radix 3 is not a power of two
    assert ws(1_000_000, 4, 16, "f64") >= 4 * 1_000_000 * 8      # four fp64 intermediates after a radix-4 level
    assert ws(10, 1, 2, "f64", 8) == 0                           # fp64: radix 2 or 4 only
    small, big = ws(1_000_000, 1, 2, "f32"), ws(100_000_000, 1, 2, "f32")
    assert 0 < small <= big
    # the literal tree keeps N/2 + N/4 intermediates, the radix-16 plan only N/16
    total = 1 << 20
    tree = ws(total, 4, 64, "f32", binding.flags_radix(2, 2))
    wide = ws(total, 4, 64, "f32", binding.flags_radix(16, 16))
    assert tree >= (32 + 16) * total * 4 and wide < 8 * total * 4


def test_plan_info(binding):
    info = binding.adasum_plan_info
    assert info(100, 1, 1, "f32")["radices"] == []
    assert info(100, 1, 2, "f32")["radices"] == [2]
    assert info(100, 1, 8, "f32", binding.flags_radix(2, 2))["radices"] == [2, 2, 2]
    assert info(100, 1, 256, "f32", binding.flags_radix(16, 16))["radices"] == [16, 16]
    assert info(100, 1, 5, "f32", binding.flags_radix(4, 4))["radices"] == [4, 2]
    linear = 1 << 18
    assert info(100, 1, 20, "f32", linear)["radices"] == [32]
    assert info(100, 1, 64, "bf16", linear)["radices"] == [64]
    with pytest.raises(binding.AdasumError):
        info(100, 1, 33, "f32", linear)                      # needs a 64 x 64 Gram matrix of fp32 inputs
    with pytest.raises(binding.AdasumError):
        info(100, 1, 8, "f32", linear | binding.flags_radix(8, 0))
    assert info(0, 0, 4, "f32")["launches"] == 0
    assert info(100, 1, 8, "f32", binding.flags_radix(2, 2))["launches"] == 4      # pass 1, two fused kernels, pass 2
    assert info(100, 1, 8, "f32", binding.flags_radix(2, 2) | (1 << 21))["launches"] == 6
    assert info(100, 1, 8, "f32", binding.flags_radix(2, 2) | (1 << 17))["launches"] == 9
    assert info(100, 1, 64, "f16")["radices"] == [64]
    assert info(100, 1, 64, "f16", 1 << 19)["radices"] == [32, 2]
    assert info(100, 1, 48, "f16")["radices"] == [32, 2]
    assert info(100, 1, 64, "f16", 1 << 19)["launches"] == 4
    assert info(100, 1, 64, "f16", (1 << 17) | (1 << 19))["launches"] == 4 + 3
    assert info(100, 1, 256, "f32")["radices"] == [16, 16]
    # fp64 buffers: levels of radix 2 or 4, two launches each
    assert info(100, 1, 64, "f64")["radices"] == [4, 4, 4]
    assert info(100, 1, 64, "f64")["launches"] == 6
    assert info(100, 1, 5, "f64", binding.flags_radix(2, 0))["radices"] == [2, 2, 2]
    for bad in (binding.flags_radix(8, 0), 1 << 18, 1 << 20, 1 << 17):
        with pytest.raises(binding.AdasumError):
            info(100, 1, 8, "f64", bad)


def _call_reduce(binding, ptrs, offsets, n, dtype=0, out=0x10000000, ws=0x20000000, ws_bytes=1 << 40, flags=0,
                 grads_null=False):
    lib = binding.raw()
    arr = (ctypes.c_void_p * max(len(ptrs), 1))(*ptrs)
    offs = np.asarray(offsets, dtype=np.int64)
    return lib.adasum_reduce(None if grads_null else arr, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                             len(offsets) - 1, n, dtype, out, ws, ws_bytes, flags, None)


def test_argument_errors_are_caught_on_the_host(binding):
    """Pointers here are made-up device addresses: every check below must fail before any CUDA
    call, so nothing is dereferenced or launched."""
    s = binding.adasum_status_string
    good = [0x30000000, 0x40000000]
    assert s(_call_reduce(binding, good, [0, 8], 2, grads_null=True)) == "ADASUM_ERR_NULL"
    assert s(_call_reduce(binding, good, [0, 8], 0)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 5000)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 2, dtype=9)) == "ADASUM_ERR_DTYPE"
    assert s(_call_reduce(binding, good, [1, 8], 2)) == "ADASUM_ERR_OFFSETS"
    assert s(_call_reduce(binding, good, [0, 8, 4], 2)) == "ADASUM_ERR_OFFSETS"
    assert s(_call_reduce(binding, good, [0, 8], 2, flags=3)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 2, flags=1 << 23)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 2, flags=64)) == "ADASUM_ERR_ARG"        # radix 64 needs 16-bit inputs
    assert s(_call_reduce(binding, [0x30000000, 0], [0, 8], 2)) == "ADASUM_ERR_NULL"
    assert s(_call_reduce(binding, good, [0, 8], 2, out=0)) == "ADASUM_ERR_NULL"
    assert s(_call_reduce(binding, good, [0, 8], 2, out=0x10000002)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, [0x30000000, 0x40000002], [0, 8], 2)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 2, ws=0)) == "ADASUM_ERR_WORKSPACE"
    assert s(_call_reduce(binding, good, [0, 8], 2, ws_bytes=16)) == "ADASUM_ERR_WORKSPACE"
    assert s(_call_reduce(binding, good, [0, 8], 2, ws=0x20000010)) == "ADASUM_ERR_ARG"
    assert s(_call_reduce(binding, good, [0, 8], 2, out=0x30000010)) == "ADASUM_ERR_ARG"      # out inside grads[0]
    assert s(_call_reduce(binding, good, [0, 8], 2, ws=0x10000000, ws_bytes=4096)) == "ADASUM_ERR_ARG"
    assert "workspace" in binding.adasum_last_error()
    # an empty reduce is fine and launches nothing
    assert s(_call_reduce(binding, good, [0, 0, 0], 2)) == "ADASUM_OK"
    assert binding.adasum_last_error() == ""


def test_shutdown_without_tables_is_ok(binding):
    binding.adasum_shutdown()


def test_package_fails_loudly_without_the_library(tmp_path, monkeypatch):
    """The product path has no fallback: with the native library absent the binding refuses to
    import."""
    import importlib.util
    import shutil

    pkg = tmp_path / "paper_2006_02924_b200"
    pkg.mkdir()
    src = os.path.join(ROOT, "paper_2006_02924_b200")
    for name in ("__init__.py", "binding.py"):
        shutil.copy(os.path.join(src, name), pkg / name)
    spec = importlib.util.spec_from_file_location("binding_without_lib", pkg / "binding.py")
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError, match="native library"):
        spec.loader.exec_module(mod)


def test_scaled_reduce_argument_errors_are_caught_on_the_host(binding):
    """adasum_reduce_scaled: a missing or misaligned scale table, a single worker and fp64 buffers
    are refused before any CUDA call (the pointers are made-up device addresses)."""
    lib = binding.raw()
    s = binding.adasum_status_string
    good = (ctypes.c_void_p * 2)(0x30000000, 0x40000000)
    offs = np.array([0, 8], dtype=np.int64)

    def call(scales=0x50000000, n=2, dtype=0):
        return lib.adasum_reduce_scaled(good, scales, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), 1, n, dtype,
                                        0x10000000, None, 0x20000000, 1 << 40, 0, None)

    assert s(call(scales=None)) == "ADASUM_ERR_NULL"
    assert "scales" in binding.adasum_last_error()
    assert s(call(scales=0x50000002)) == "ADASUM_ERR_ARG"
    assert s(call(n=1)) == "ADASUM_ERR_ARG"
    assert s(call(dtype=3)) == "ADASUM_ERR_DTYPE"
