"""Build libtopoep.so in-tree with nvcc for sm_100a (no torch involved)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtopoep.so")
SOURCES = ["api.cu", "hist.cu", "hist_static.cu", "solve.cu", "route.cu", "reroute.cu", "plan_tail.cu", "dispatch.cu", "transfer.cu", "summary.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-shared"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "topoep.h"))
    return any(os.path.getmtime(d) > t for d in deps)


CHECKED_LIB = os.path.join(HERE, "libtopoep_checked.so")


def build_checked(force: bool = False) -> str:
    """The bounds-checked build (tests only): every index that is derived from data is checked,
    an index out of range sets TOPOEP_FLAG_INTERNAL and is clamped.  A library of its own."""
    if not force and os.path.exists(CHECKED_LIB) and not _stale(CHECKED_LIB):
        return CHECKED_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = CHECKED_LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + ["-DTOPOEP_CHECKED", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, CHECKED_LIB)
    return CHECKED_LIB


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source into one shared library next to this file."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    extra = os.environ.get("TOPOEP_NVCC_EXTRA", "").split()   # e.g. -D switches while tuning
    cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
