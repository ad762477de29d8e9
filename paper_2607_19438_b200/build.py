"""Builds the C-ABI CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libqgemm_b200.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo", "-shared",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default", "--expt-relaxed-constexpr"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(HERE, "..", "include", "qgemm.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + sources()
        subprocess.check_call(cmd)
    return LIB


PROFILE_LIB = os.path.join(HERE, "libqgemm_b200_prof.so")


def build_profile(force: bool = False) -> str:
    """The same library with -DQG_PROFILE: the GEMM kernel's roles add up the cycles they spend in each of their waits
    (read back with qg_debug_set_stats).  Slower than the product build; used by `bench.py --case roles` only."""
    if force or not os.path.exists(PROFILE_LIB) or os.path.getmtime(PROFILE_LIB) < os.path.getmtime(build()):
        subprocess.check_call([NVCC] + FLAGS + ["-DQG_PROFILE", "-o", PROFILE_LIB] + sources())
    return PROFILE_LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
    if "--profile" in sys.argv:
        print(build_profile(force=True))
