"""Builds libsonic.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsonic.so")
SOURCES = ["sonic.cu"]
HEADERS = ["sonic_common.cuh", "sonic_dense.cuh", "sonic_stream.cuh", "sonic_exact.cuh", "../../include/sonic.h"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.exists(d) and os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared",
           "-o", LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return LIB


WAITTEST_LIB = os.path.join(HERE, "libsonic_waittest.so")


def build_waittest(force: bool = False) -> str:
    """The test-only variant used by tests/test_gpu_wait_expiry.py: bounded waits give up after 4096 rounds and a
    header word lets a test withhold one tile's copy, so that a wait really runs out (no fault, no hang)."""
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    if not force and os.path.exists(WAITTEST_LIB) and all(os.path.getmtime(d) <= os.path.getmtime(WAITTEST_LIB) for d in deps if os.path.exists(d)):
        return WAITTEST_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-DSONIC_TEST_WITHHOLD", "-DSONIC_WAIT_LIMIT=4096u",
           "-o", WAITTEST_LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    return WAITTEST_LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
