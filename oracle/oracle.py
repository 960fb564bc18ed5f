"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this module. It compiles ``hccl_oracle.c`` with gcc on first use and exposes
each C function on numpy arrays. Rank buffers are lists of 1-D numpy arrays:
``float32`` for fp32 data, ``uint16`` raw bit patterns for bf16/fp16 data, and
``uint8`` for the byte-level AllToAllv/AllGather calls.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

FP32, BF16, FP16 = 0, 1, 2
_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hccl_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FP contraction). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def np_dtype(dt: int):
    return np.float32 if dt == FP32 else np.uint16


def _ptrs(bufs, writable=False):
    arr = (ctypes.c_void_p * len(bufs))()
    for i, b in enumerate(bufs):
        assert isinstance(b, np.ndarray) and b.flags["C_CONTIGUOUS"]
        if writable:
            assert b.flags["WRITEABLE"]
        arr[i] = b.ctypes.data
    return arr


def _i64(a):
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _check(rc, what):
    if rc != 0:
        raise ValueError("oracle: invalid arguments to " + what)


def widen(dt: int, a: np.ndarray) -> np.ndarray:
    out = np.empty(a.size, dtype=np.float64)
    lib().oracle_widen(ctypes.c_int(dt), ctypes.c_int64(a.size), ctypes.c_void_p(a.ctypes.data),
                       ctypes.c_void_p(out.ctypes.data))
    return out


def round_to(dt: int, a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float64)
    out = np.empty(a.size, dtype=np_dtype(dt))
    lib().oracle_round(ctypes.c_int(dt), ctypes.c_int64(a.size), ctypes.c_void_p(a.ctypes.data),
                       ctypes.c_void_p(out.ctypes.data))
    return out


def nmc(dt_dst: int, dt_a: int, a: np.ndarray, dt_b: int | None = None, b: np.ndarray | None = None):
    """dst = round(f32(a) + f32(b)); with b None: dst = a (copy form)."""
    n = a.size
    out = np.empty(n, dtype=np_dtype(dt_dst))
    rc = lib().oracle_nmc(ctypes.c_int(dt_dst), ctypes.c_void_p(out.ctypes.data), ctypes.c_int(dt_a),
                          ctypes.c_void_p(a.ctypes.data), ctypes.c_int(dt_b if b is not None else dt_a),
                          ctypes.c_void_p(b.ctypes.data if b is not None else None), ctypes.c_int64(n))
    _check(rc, "nmc")
    return out


def allreduce(dt: int, X: list) -> list:
    R, n = len(X), X[0].size
    Y = [np.empty(n, dtype=np_dtype(dt)) for _ in range(R)]
    _check(lib().oracle_allreduce(R, ctypes.c_int64(n), dt, _ptrs(X), _ptrs(Y, True)), "allreduce")
    return Y


def reducescatter(dt: int, X: list, recvcounts) -> list:
    R = len(X)
    rc, rcp = _i64(recvcounts)
    assert int(rc.sum()) == X[0].size
    Y = [np.empty(int(rc[r]), dtype=np_dtype(dt)) for r in range(R)]
    _check(lib().oracle_reducescatter(R, rcp, dt, _ptrs(X), _ptrs(Y, True)), "reducescatter")
    return Y


def allgatherv(X: list) -> list:
    """X: per-rank 1-D arrays of one dtype; returns R copies of their concatenation."""
    R = len(X)
    counts, cp = _i64([x.size for x in X])
    Y = [np.empty(int(counts.sum()), dtype=X[0].dtype) for _ in range(R)]
    _check(lib().oracle_allgatherv(R, cp, X[0].dtype.itemsize, _ptrs(X), _ptrs(Y, True)), "allgatherv")
    return Y


def packed_displs(sendcounts):
    C, cp = _i64(sendcounts)
    R = C.shape[0]
    sd = np.empty((R, R), dtype=np.int64)
    rd = np.empty((R, R), dtype=np.int64)
    lib().oracle_packed_displs(R, cp, sd.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                               rd.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
    return sd, rd


def alltoallv(X: list, Y: list, sendcounts, sdispls, rdispls, row_bytes: int, dst_only: int = -1):
    """Writes into the caller's Y (uint8 arrays), so untouched bytes stay as the caller left them."""
    R = len(X)
    C, cp = _i64(sendcounts)
    SD, sp = _i64(sdispls)
    RD, rp = _i64(rdispls)
    rc = lib().oracle_alltoallv(R, cp, sp, rp, ctypes.c_int64(row_bytes), _ptrs(X), _ptrs(Y, True),
                                ctypes.c_int(dst_only))
    _check(rc, "alltoallv")
    return Y


def _ring(fn, dt, X, offs_or_counts, nout):
    R = len(X)
    a, ap = _i64(offs_or_counts)
    Y = [np.empty(nout(r), dtype=np_dtype(dt)) for r in range(R)]
    _check(fn(R, ap, dt, _ptrs(X), _ptrs(Y, True)), "ring")
    return Y


def allreduce_ring_f32(dt: int, X: list, offs) -> list:
    n = X[0].size
    return _ring(lib().oracle_allreduce_ring_f32, dt, X, offs, lambda r: n)


def reducescatter_ring_f32(dt: int, X: list, recvcounts) -> list:
    rc = np.asarray(recvcounts, dtype=np.int64)
    return _ring(lib().oracle_reducescatter_ring_f32, dt, X, rc, lambda r: int(rc[r]))


def bidirectional_segments(n: int, R: int, granule: int):
    """Chunk c (floor split of n over R) cut into granules; granule k of a chunk travels forwards when k is
    even and backwards when k is odd. Returns (seg_off [nseg+1], seg_chunk, seg_dir)."""
    offs = floor_chunk_offsets(n, R)
    off, chunk, direction = [], [], []
    for c in range(R):
        lo, hi = int(offs[c]), int(offs[c + 1])
        k = 0
        while lo < hi:
            off.append(lo)
            chunk.append(c)
            direction.append(1 if k % 2 == 0 else -1)
            lo = min(hi, lo + granule)
            k += 1
    off.append(n)
    return np.array(off, dtype=np.int64), np.array(chunk, dtype=np.int64), np.array(direction, dtype=np.int64)


def allreduce_ring_dir_f32(dt: int, X: list, seg_off, seg_chunk, seg_dir) -> list:
    R, n = len(X), X[0].size
    so, sop = _i64(seg_off)
    sc, scp = _i64(seg_chunk)
    sd, sdp = _i64(seg_dir)
    Y = [np.empty(n, dtype=np_dtype(dt)) for _ in range(R)]
    _check(lib().oracle_allreduce_ring_dir_f32(R, int(sc.size), sop, scp, sdp, dt, _ptrs(X), _ptrs(Y, True)), "ring_dir")
    return Y


def two_level_offsets(n: int, G: int, L: int):
    """Chunk j of L (floor split of n), each cut into G sub-chunks (floor split of the chunk)."""
    offs1 = floor_chunk_offsets(n, L)
    offs2 = np.zeros((L, G + 1), dtype=np.int64)
    for j in range(L):
        lo, hi = int(offs1[j]), int(offs1[j + 1])
        offs2[j] = [lo + (k * (hi - lo)) // G for k in range(G + 1)]
    return offs1, offs2


def allreduce_ring2_f32(dt: int, X: list, G: int, L: int) -> list:
    R, n = len(X), X[0].size
    assert R == G * L
    offs1, offs2 = two_level_offsets(n, G, L)
    o1, p1 = _i64(offs1)
    o2, p2 = _i64(offs2)
    Y = [np.empty(n, dtype=np_dtype(dt)) for _ in range(R)]
    _check(lib().oracle_allreduce_ring2_f32(G, L, p1, p2, dt, _ptrs(X), _ptrs(Y, True)), "ring2")
    return Y


def allreduce_oneshot_f32(dt: int, X: list) -> list:
    R, n = len(X), X[0].size
    Y = [np.empty(n, dtype=np_dtype(dt)) for _ in range(R)]
    _check(lib().oracle_allreduce_oneshot_f32(R, ctypes.c_int64(n), dt, _ptrs(X), _ptrs(Y, True)), "oneshot")
    return Y


def allreduce_tree_f32(dt: int, X: list) -> list:
    R, n = len(X), X[0].size
    Y = [np.empty(n, dtype=np_dtype(dt)) for _ in range(R)]
    _check(lib().oracle_allreduce_tree_f32(R, ctypes.c_int64(n), dt, _ptrs(X), _ptrs(Y, True)), "tree")
    return Y


def ulp_distance(dt: int, a: np.ndarray, b: np.ndarray) -> np.ndarray:
    assert a.size == b.size and a.dtype == b.dtype
    out = np.empty(a.size, dtype=np.int64)
    lib().oracle_ulp_distance(dt, ctypes.c_int64(a.size), ctypes.c_void_p(a.ctypes.data),
                              ctypes.c_void_p(b.ctypes.data), ctypes.c_void_p(out.ctypes.data))
    return out


def sum_f64(dt: int, X: list) -> np.ndarray:
    R, n = len(X), X[0].size
    out = np.empty(n, dtype=np.float64)
    _check(lib().oracle_sum_f64(R, ctypes.c_int64(n), dt, _ptrs(X), ctypes.c_void_p(out.ctypes.data)), "sum_f64")
    return out


def floor_chunk_offsets(n: int, R: int) -> np.ndarray:
    """Chunk c of an n-element buffer split R ways covers [floor(c n / R), floor((c+1) n / R))."""
    return np.array([(c * n) // R for c in range(R + 1)], dtype=np.int64)
