"""Builds csrc/*.cu into libmosaic_bsa.so (in-tree) with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmosaic_bsa.so")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", INCLUDE, "-I", CSRC, "-o", tmp] + sources()
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


WAIT_TEST_LIB = os.path.join(os.path.dirname(HERE), "tests", "libmosaic_bsa_waittest.so")


def build_wait_test(force: bool = False) -> str:
    """Test-only variant of the library (never loaded by the product): waits are bounded by about a millisecond
    and the planner of the tensor-core kernels never publishes a CTA's first key list, so that every consumer's
    wait runs out and the kernels' time-out path (status word, orderly exit) can be exercised without a fault.
    It also carries a tiny probe kernel that waits on a barrier nothing arrives at."""
    probe = os.path.join(os.path.dirname(HERE), "tests", "cuda", "wait_probe.cu")
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h")) + [probe]
    if not force and os.path.exists(WAIT_TEST_LIB) and all(os.path.getmtime(d) <= os.path.getmtime(WAIT_TEST_LIB) for d in deps):
        return WAIT_TEST_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = WAIT_TEST_LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-DMOSAIC_TEST_SPIN_CYCLES=2000000ll", "-DMOSAIC_TEST_WITHHOLD_FIRST_LIST=1",
           "-Xcompiler", "-fPIC", "-shared", "-I", INCLUDE, "-I", CSRC, "-o", tmp] + sources() + [probe]
    subprocess.check_call(cmd)
    os.replace(tmp, WAIT_TEST_LIB)
    return WAIT_TEST_LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
