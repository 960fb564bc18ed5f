"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers and lays them out; it contains none of the
collectives' arithmetic (no sums, no displacement rules, no rounding of results)
so the CUDA path's tests and the CPU oracle's tests can both be fed from it.

The shapes follow what the paper says about its workloads (Sec. I, Sec. V-A):
large AllToAllv exchanges of embedding rows with irregular per-peer splits,
AllReduce/ReduceScatter of gradient-like tensors, rack-sized groups of 16 and
jobs of 64+ ranks, and small latency-bound AllReduce messages for inference
(Sec. IV-B). Production traces are not available; these stand in for them.

16-bit floating-point data is carried as raw ``uint16`` bit patterns.
"""
from __future__ import annotations

import numpy as np
import torch

FP32, BF16, FP16 = 0, 1, 2
ELEM_BYTES = {FP32: 4, BF16: 2, FP16: 2}


def to_bits(x: np.ndarray, dt: int) -> np.ndarray:
    """Store float32 samples as the given element type (library conversion, nearest-even)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dt == FP32:
        return x
    if dt == FP16:
        return x.astype(np.float16).view(np.uint16)
    t = torch.from_numpy(x).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def from_bits(a: np.ndarray, dt: int) -> np.ndarray:
    """Bit patterns -> float64 values by library routines (for test-side checks only)."""
    if dt == FP32:
        return a.astype(np.float64)
    if dt == FP16:
        return a.view(np.float16).astype(np.float64)
    t = torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def uniform_ranks(R: int, n: int, dt: int, seed: int, lo=-1.0, hi=1.0) -> list:
    """R rank buffers of n values uniform in [lo, hi) (config: ring AllReduce of fp32 gradients)."""
    rng = np.random.default_rng(seed)
    return [to_bits(rng.uniform(lo, hi, size=n).astype(np.float32), dt) for _ in range(R)]


def normal_ranks(R: int, n: int, dt: int, seed: int, std=1.0) -> list:
    """R rank buffers of n values ~ N(0, std^2) (gradient-like for std=0.02; activations for std=1)."""
    rng = np.random.default_rng(seed)
    return [to_bits((rng.standard_normal(size=n) * std).astype(np.float32), dt) for _ in range(R)]


def small_int_ranks(R: int, n: int, dt: int, seed: int, span=8) -> list:
    """Small integers: every partial sum is exact in every element type, so results are unique."""
    rng = np.random.default_rng(seed)
    return [to_bits(rng.integers(-span, span + 1, size=n).astype(np.float32), dt) for _ in range(R)]


def uniform_counts(R: int, seed: int, hi: int = 4096) -> np.ndarray:
    """R x R per-(source, destination) row counts, uniform in [0, hi]."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, hi + 1, size=(R, R), dtype=np.int64)


def zipf_counts(R: int, seed: int, s: float = 1.1, cap: int = 32768) -> np.ndarray:
    """Heavily skewed R x R row counts: Zipf(s) draws (support >= 1) clamped at cap."""
    rng = np.random.default_rng(seed)
    return np.minimum(rng.zipf(s, size=(R, R)), cap).astype(np.int64)


# ---- regenerable row payloads -------------------------------------------------
# A row's 16-bit words are a hash of (source rank, row index, column), so any row
# of any rank can be produced again, on the host or on the device, without
# keeping the whole send buffer. Words whose fp16 exponent field is all ones are
# changed so every word is a finite fp16 (and bf16) value.
_M1, _M2, _M3, _M4 = 0x5BD1E995, 0x2C1B3C6D, 0x297A2D39, 0x1B873593  # all < 2**31


def _mix(xp, src, row, col):
    m32 = 0xFFFFFFFF
    h = (row * _M1 + col * _M2 + src * _M3 + 0x3C6EF372) & m32
    h = h ^ (h >> 15)
    h = (h * _M4) & m32
    h = h ^ (h >> 13)
    h = (h * _M1) & m32
    h = h ^ (h >> 16)
    w = h & 0xFFFF
    bad = (w & 0x7C00) == 0x7C00
    w = xp.where(bad, w ^ 0x4000, w)
    return w


def hashed_rows_np(src: int, row0: int, nrows: int, row_elems: int) -> np.ndarray:
    """uint16 [nrows, row_elems]: rows row0 .. row0+nrows-1 of source rank src."""
    row = np.arange(row0, row0 + nrows, dtype=np.int64)[:, None]
    col = np.arange(row_elems, dtype=np.int64)[None, :]
    return _mix(np, np.int64(src), row, col).astype(np.uint16)


def hashed_rows_torch(src: int, row0: int, nrows: int, row_elems: int, device) -> torch.Tensor:
    """int16 [nrows, row_elems] on device, bit-identical to hashed_rows_np."""
    row = torch.arange(row0, row0 + nrows, dtype=torch.int64, device=device)[:, None]
    col = torch.arange(row_elems, dtype=torch.int64, device=device)[None, :]
    w = _mix(torch, src, row, col)
    return w.to(torch.int16)


def fill_hashed_rows_torch(out: torch.Tensor, src: int, row_elems: int, block_rows: int = 1 << 16):
    """Fill a device int16 buffer of whole rows block by block (bounded temporaries)."""
    nrows = out.numel() // row_elems
    v = out.view(nrows, row_elems)
    for r0 in range(0, nrows, block_rows):
        nb = min(block_rows, nrows - r0)
        v[r0:r0 + nb] = hashed_rows_torch(src, r0, nb, row_elems, out.device)
    return out
