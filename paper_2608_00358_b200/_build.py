"""Builds the C-ABI library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libhccl_b200.so")
# one translation unit per kernel, so that they compile in parallel (each takes about a minute)
SOURCES = ["graph.cpp", "collectives.cpp", "verify.cpp", "executor.cu", "kernel_lsu.cu", "kernel_lsu_light.cu", "kernel_bulk.cu",
           "kernel_resident.cu", "kernel_chain.cu"]
HEADERS = ["plan.hpp", "tables.h", "device.cuh", "bulk.cuh", "bulk_layout.h", "kernels.cuh", os.path.join("..", "..", "include", "hccl.h")]
# a kernel's unit does not use every helper of the shared headers: no "declared but never referenced" remarks for them
QUIET = ["-diag-suppress", "177"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    files = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(f) > t for f in files)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/ into libhccl_b200.so next to this file. Returns the library path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    jobs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, os.path.splitext(src)[0] + ".o")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (QUIET if src.endswith(".cu") else []) + \
            ["-x", "cu", "-c", os.path.join(CSRC, src), "-o", obj]
        jobs.append((cmd, obj))
    procs = [(subprocess.Popen(cmd), cmd) for cmd, _ in jobs]
    failed = [cmd for pr, cmd in procs if pr.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, failed[0])
    objs = [obj for _, obj in jobs]
    tmp = LIB + ".%d.tmp" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
