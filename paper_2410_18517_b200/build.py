"""Compile the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libkvs.so")
# the same sources with -DKVS_DEBUG_BOUNDS: every computed global offset is checked on the device
LIB_BOUNDS = os.path.join(HERE, "libkvs_bounds.so")
# the same sources with -DKVS_TRACE: the attention kernels stamp a per-block timeline (kvs_trace_begin)
LIB_TRACE = os.path.join(HERE, "libkvs_trace.so")
SOURCES = ["kvs_api.cu", "kvs_kernels.cu", "kvs_mma.cu", "kvs_prefill.cu", "kvs_prefill_f32.cu", "kvs_search.cu"]
HEADERS = ["kvs_device.cuh", "kvs_kernels.h", os.path.join("..", "..", "include", "kvs.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, bounds: bool = False, trace: bool = False) -> str:
    """Build ``libkvs.so`` (or, with ``bounds``, the bounds-checking ``libkvs_bounds.so``; with ``trace``, the
    timeline-stamping ``libkvs_trace.so``) next to this file if it is missing or older than its sources."""
    lib = LIB_BOUNDS if bounds else (LIB_TRACE if trace else LIB)
    if not force and not is_stale(lib):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (["-DKVS_DEBUG_BOUNDS"] if bounds else []) + (["-DKVS_TRACE"] if trace and not bounds else [])
    cmd += ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, bounds="--bounds" in sys.argv,
                trace="--trace" in sys.argv))
