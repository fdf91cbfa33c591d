"""Builds libbr.so (the C-ABI routing library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbr.so")
LIB_DEBUG = os.path.join(HERE, "libbr_dbg.so")          # the same sources with range-checked indexing (-DBR_BOUNDS)
SOURCES = ["br_api.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false",                       # scores are evaluated term by term, never contracted
    "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-ffp-contract=off",
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    # every file of csrc/ is a dependency: the kernels live in headers included by br_api.cu
    deps = glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cuh"))
    deps.append(os.path.join(os.path.dirname(HERE), "include", "br.h"))
    deps.append(os.path.abspath(__file__))
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(lib: str, extra, verbose: bool) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lcudart"]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        _compile(LIB, [], verbose)
    return LIB


def build_all(force: bool = False) -> None:
    """Both libraries, compiled side by side when both are out of date."""
    import threading
    jobs = []
    if force or _stale():
        jobs.append(threading.Thread(target=_compile, args=(LIB, [], False)))
    if force or _stale(LIB_DEBUG):
        jobs.append(threading.Thread(target=_compile, args=(LIB_DEBUG, ["-DBR_BOUNDS"], False)))
    for j in jobs:
        j.start()
    for j in jobs:
        j.join()
    if not (os.path.exists(LIB) and os.path.exists(LIB_DEBUG)):
        raise RuntimeError("building the CUDA libraries failed (see the compiler output above)")


def build_debug(force: bool = False) -> str:
    """The range-checked library: every index into a per-instance array is checked and counted."""
    if force or _stale(LIB_DEBUG):
        _compile(LIB_DEBUG, ["-DBR_BOUNDS"], False)
    return LIB_DEBUG


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv))
