"""Builds the native library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2006_02924_b200.build [--force] [--verbose]

Every .cu file under csrc/ is a translation unit of its own; they are compiled in parallel and
linked into one shared library.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB_DIR = os.path.join(PKG, "lib")
OBJ_DIR = os.path.join(PKG, "_build")
LIB_PATH = os.path.join(LIB_DIR, "libadasum_b200.so")
SOURCES = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) +
                 [os.path.join(ROOT, "include", "adasum.h")])
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _object_of(source: str) -> str:
    return os.path.join(OBJ_DIR, os.path.splitext(os.path.basename(source))[0] + ".o")


def _newer_than(target: str, deps) -> bool:
    if not os.path.exists(target):
        return False
    built = os.path.getmtime(target)
    return all(os.path.getmtime(p) <= built for p in deps)


def up_to_date() -> bool:
    return _newer_than(LIB_PATH, SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles what is out of date and returns the library's path.  Prints one line saying
    whether anything was compiled."""
    if not force and up_to_date():
        print(f"[build] {os.path.relpath(LIB_PATH, ROOT)} is up to date: nothing compiled")
        return LIB_PATH
    os.makedirs(LIB_DIR, exist_ok=True)
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    stale = [s for s in SOURCES if force or not _newer_than(_object_of(s), [s] + HEADERS)]

    def compile_one(source: str) -> None:
        cmd = [nvcc, *ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-c",
               "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", _object_of(source), source]
        if verbose:
            cmd += ["-Xptxas", "-v"]
        subprocess.check_call(cmd)

    with ThreadPoolExecutor(max_workers=max(1, min(len(stale), os.cpu_count() or 1))) as pool:
        list(pool.map(compile_one, stale))
    tmp = LIB_PATH + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, *ARCH, "-shared", "-Xcompiler", "-fPIC", "-o", tmp, *[_object_of(s) for s in SOURCES]])
    os.replace(tmp, LIB_PATH)
    print(f"[build] compiled {', '.join(os.path.basename(s) for s in stale)} with {nvcc} for sm_100a "
          f"-> {os.path.relpath(LIB_PATH, ROOT)}")
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
