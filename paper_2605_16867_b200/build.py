"""Builds libgoodserve.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libgoodserve.so")
COUNT_LIB_PATH = os.path.join(_PKG, "libgoodserve_count.so")    # the measuring build (-DGS_COUNT_EVALS)
DEBUG_LIB_PATH = os.path.join(_PKG, "libgoodserve_debug.so")    # the checking build (-DGS_DEBUG)
SOURCES = ("api.cu", "prologue.cu", "route.cu", "risk.cu", "sequential.cu")
NVCC_FLAGS = ("-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--shared",
              "-cudart", "shared")


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libgoodserve.so cannot be built")


def _stale(path: str) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "goodserve.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), counting: bool = False,
                  checking: bool = False) -> str:
    """Builds libgoodserve.so, or with ``counting`` the measuring build whose work counters tick,
    or with ``checking`` the build whose table index checks are compiled in."""
    path = COUNT_LIB_PATH if counting else DEBUG_LIB_PATH if checking else LIB_PATH
    if not force and not _stale(path):
        return path
    if counting:
        extra_flags = (*extra_flags, "-DGS_COUNT_EVALS")
    elif checking:
        extra_flags = (*extra_flags, "-DGS_DEBUG")
    cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, "-I", INCLUDE, "-I", CSRC,
           *[os.path.join(CSRC, s) for s in SOURCES], "-o", path + ".tmp"]
    if verbose:
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(path + ".tmp", path)
    return path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True,
                        extra_flags=("-Xptxas", "-v") if "--ptxas" in sys.argv else ()))
    if "--counting" in sys.argv:
        print(build_library(force="--force" in sys.argv, verbose=True, counting=True))
    if "--checking" in sys.argv:
        print(build_library(force="--force" in sys.argv, verbose=True, checking=True))
