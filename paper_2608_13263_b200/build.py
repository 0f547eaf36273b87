"""Builds the CUDA library in-tree with nvcc for sm_100a:

  libvtoken.so          the repack library (C ABI of include/vtoken.h)
  libvtoken_checked.so  the same sources with -DVTOKEN_CHECKED: every index into scratch, tables and pools
                        range-checked (an out-of-range access is skipped and flagged, never a fault), and the
                        stall hook of the time-out test; used by the tests in place of a memory sanitizer

``python -m paper_2608_13263_b200.build`` rebuilds when a source is newer than its library.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")

LIB = os.path.join(PKG, "libvtoken.so")
CHECKED_LIB = os.path.join(PKG, "libvtoken_checked.so")

LIB_SOURCES = ["api.cu", "plan.cu", "plan_small.cu", "copy.cu", "gather.cu", "gather_static.cu", "runtime.cu", "plan_partial.cu",
               "waves.cu", "slot_cache.cu", "check.cu"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC",
              "-cudart", "static"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA libraries cannot be built")


def _stale(lib: str, sources) -> bool:
    if not os.path.exists(lib):
        return True
    deps = [os.path.join(CSRC, s) for s in sources] + [os.path.join(CSRC, "common.cuh"),
                                                       os.path.join(INCLUDE, "vtoken.h")]
    return os.path.getmtime(lib) < max(os.path.getmtime(d) for d in deps if os.path.exists(d))


def _build(lib: str, sources, verbose: bool, extra=()) -> None:
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-I", INCLUDE, "-I", CSRC, "-o", tmp] + [os.path.join(CSRC, s) for s in sources]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> None:
    if force or _stale(LIB, LIB_SOURCES):
        _build(LIB, LIB_SOURCES, verbose)
    if force or _stale(CHECKED_LIB, LIB_SOURCES):
        _build(CHECKED_LIB, LIB_SOURCES, verbose, extra=["-DVTOKEN_CHECKED"])


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
