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


def _nvcc_cmd(out: str, defines=(), verbose: bool = False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared"] + list(defines) + ["-o", out] + [os.path.join(CSRC, f) for f in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    return cmd


def _fresh(lib: str) -> bool:
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return os.path.exists(lib) and all(os.path.getmtime(d) <= os.path.getmtime(lib) for d in deps if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    subprocess.run(_nvcc_cmd(LIB, verbose=verbose), check=True)
    return LIB


# Two variants of the same sources, never loaded by the product path:
#  * libsonic_waittest.so (tests/test_gpu_wait_expiry.py): bounded waits give up after 4096 rounds and a header word lets
#    a test withhold one tile's copy, so that a wait really runs out (no fault, no hang);
#  * libsonic_trace.so (bench.py --timeline): every kernel leaves its earliest start and latest end (globaltimer) in the
#    workspace header.
WAITTEST_LIB = os.path.join(HERE, "libsonic_waittest.so")
TRACE_LIB = os.path.join(HERE, "libsonic_trace.so")
VARIANTS = {WAITTEST_LIB: ("-DSONIC_TEST_WITHHOLD", "-DSONIC_WAIT_LIMIT=4096u"), TRACE_LIB: ("-DSONIC_TRACE",)}


def build_waittest(force: bool = False) -> str:
    if force or not _fresh(WAITTEST_LIB):
        subprocess.run(_nvcc_cmd(WAITTEST_LIB, VARIANTS[WAITTEST_LIB]), check=True)
    return WAITTEST_LIB


def build_trace(force: bool = False) -> str:
    if force or not _fresh(TRACE_LIB):
        subprocess.run(_nvcc_cmd(TRACE_LIB, VARIANTS[TRACE_LIB]), check=True)
    return TRACE_LIB


def build_all(force: bool = False) -> None:
    """The library and its two variants, compiled side by side."""
    jobs = []
    if force or _stale():
        jobs.append(subprocess.Popen(_nvcc_cmd(LIB)))
    for lib, defs in VARIANTS.items():
        if force or not _fresh(lib):
            jobs.append(subprocess.Popen(_nvcc_cmd(lib, defs)))
    bad = [j.args for j in jobs if j.wait() != 0]
    if bad:
        raise RuntimeError("nvcc failed: %s" % bad)


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
