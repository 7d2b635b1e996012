"""Compiles the CUDA library in-tree for sm_100a.  Run as ``python -m paper_2607_22614_b200.build``."""
from __future__ import annotations

import os
import subprocess
import sys

_DIR = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_DIR)
CSRC = os.path.join(_DIR, "csrc")
LIB = os.path.join(_DIR, "libdynaresize.so")
SOURCES = ["api.cu", "planner.cpp", "copy_pool.cpp", "reshard.cu", "staging.cu", "stream.cu", "quant.cu", "probe.cu", "controller.cpp"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC,-Wall,-pthread"]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_ROOT, "include", "dynaresize.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or stale()):
        return LIB
    # DR_NVCC_FLAGS adds flags, e.g. the kernels' compile-time options (-DDR_BULK_STORE=1, -DDR_BULK=0, ...)
    extra = os.environ.get("DR_NVCC_FLAGS", "").split()
    cmd = ["nvcc", *NVCC_FLAGS, *extra, "-I", os.path.join(_ROOT, "include"), "-I", CSRC, "-shared", "-o", LIB,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
