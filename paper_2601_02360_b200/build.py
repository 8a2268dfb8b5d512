"""Builds the CUDA library in-tree: csrc/*.cu -> csrc/libsparseloco.so (sm_100a only).

  python -m paper_2601_02360_b200.build [--force] [-v]     the library
  python -m paper_2601_02360_b200.build --debug            csrc/libsparseloco_debug.so: the same sources
                                                           compiled with -DSL_DEBUG_BOUNDS (every index the
                                                           Eq. 2 kernels use is range-checked; a violation
                                                           raises SL_FLAG_BOUNDS and the access is skipped)

Sources are compiled to objects side by side (csrc/build/, git-ignored) and linked; only what
changed is recompiled.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_CSRC = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc")
LIB_PATH = os.path.join(_CSRC, "libsparseloco.so")
DEBUG_LIB_PATH = os.path.join(_CSRC, "libsparseloco_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",            # nothing may be contracted: every fused op is an explicit intrinsic
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(_CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(_CSRC, "*.cuh")) + [os.path.join(_CSRC, "..", "..", "include", "sparseloco.h")]


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not _newer(sources() + _headers(), lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    objdir = os.path.join(_CSRC, "build", "debug" if debug else "release")
    os.makedirs(objdir, exist_ok=True)
    flags = NVCC_FLAGS + (["-DSL_DEBUG_BOUNDS"] if debug else []) + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src: str) -> str:
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        if force or _newer([src] + _headers(), obj):
            tmp = obj + f".{os.getpid()}.tmp"
            subprocess.check_call([nvcc] + flags + ["-c", src, "-o", tmp])
            os.replace(tmp, obj)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(compile_one, sources()))
    tmp = lib + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
