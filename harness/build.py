"""Builds the harness kernels in-tree with nvcc for sm_100a: ``libvtoken_harness.so`` (pool
fill, whole-pool verifier, decode-read proxy).  ``python -m harness.build`` rebuilds when the
source is newer than the library."""
from __future__ import annotations

import os
import subprocess
import sys

from paper_2608_13263_b200.build import NVCC_FLAGS, _nvcc

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(HERE, "csrc", "harness.cu")
HARNESS_LIB = os.path.join(HERE, "libvtoken_harness.so")


def build(force: bool = False, verbose: bool = False) -> None:
    if not force and os.path.exists(HARNESS_LIB) and os.path.getmtime(HARNESS_LIB) >= os.path.getmtime(SOURCE):
        return
    tmp = HARNESS_LIB + f".{os.getpid()}.tmp"
    cmd = [_nvcc(), *NVCC_FLAGS, "-o", tmp, SOURCE]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.check_call(cmd)
    os.replace(tmp, HARNESS_LIB)


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
