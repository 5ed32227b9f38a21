"""Seeded synthetic inputs for the five softmax workloads.

This module serves both the CUDA library's tests/benchmark and the CPU oracle's tests. It holds
none of the softmax arithmetic: only random draws, the per-workload structure (row bias, spikes,
causal mask) and the one rounding to the stored dtype. Arrays are numpy, on the host, as stored
bit patterns: ``float32`` for fp32, ``uint16`` for bf16 and fp16.

The workloads stand in for the operator captures of the paper's Table I (LLM eager-attention
softmax, MoE router softmax), whose models and prompt sets are not available; shapes, dtypes and
value distributions are the ones the benchmark contract fixes.

Generation is counter-based per row block: block ``b`` of workload ``k`` draws from
``numpy.random.Philox(key=[seed, b])``, so any row range can be produced on its own (full-size
parity checks regenerate sampled rows without materialising the matrix) and blocks can be
produced in parallel with the same result.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

FP32, BF16, FP16 = 0, 1, 2
ELEM_SIZE = {FP32: 4, BF16: 2, FP16: 2}
DTYPE_NAME = {FP32: "fp32", BF16: "bf16", FP16: "fp16"}
NP_STORE = {FP32: np.float32, BF16: np.uint16, FP16: np.uint16}


# ---------------------------------------------------------------------------------------------
# one rounding from fp64 to the stored format
# ---------------------------------------------------------------------------------------------

def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp64 -> bfloat16 bit patterns, nearest-even, with a single rounding.

    fp64 is first narrowed to fp32 with round-to-odd (truncate, then OR the sticky bit into the
    last place); nearest-even from there to the 8-bit significand equals direct rounding because
    fp32 keeps 16 more bits than bf16.
    """
    a = np.asarray(a, dtype=np.float64)
    f = a.astype(np.float32)
    back = f.astype(np.float64)
    bits = f.view(np.uint32).copy()
    finite = np.isfinite(a)
    inexact = (back != a) & finite
    away = (np.abs(back) > np.abs(a)) & finite
    bits -= away.astype(np.uint32)          # step the magnitude back to the truncated value
    bits |= inexact.astype(np.uint32)       # sticky
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 -> bfloat16 bit patterns, nearest-even (NaN -> quiet NaN)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if np.any(nan):
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_stored(a: np.ndarray, dtype: int) -> np.ndarray:
    """Round an fp64/fp32 array once to the stored format and return its stored representation."""
    if dtype == FP32:
        return np.asarray(a).astype(np.float32)
    if dtype == BF16:
        return f64_to_bf16_bits(np.asarray(a, dtype=np.float64))
    return np.asarray(a).astype(np.float16).view(np.uint16)   # numpy narrows fp64 -> fp16 directly


def stored_to_f32(x: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == FP32:
        return np.asarray(x, dtype=np.float32)
    if dtype == BF16:
        return bf16_bits_to_f32(x)
    return np.asarray(x, dtype=np.uint16).view(np.float16).astype(np.float32)


# ---------------------------------------------------------------------------------------------
# workloads
# ---------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # 1..5
    dtype: int
    rows: int
    cols: int
    scale: float          # passed to the library as a C float
    seed: int
    block_rows: int       # rows generated per counter block
    note: str

    @property
    def elem_size(self) -> int:
        return ELEM_SIZE[self.dtype]

    @property
    def min_bytes(self) -> int:
        """Read x once + write y once."""
        return 2 * self.rows * self.cols * self.elem_size

    @property
    def scale_f32(self) -> float:
        return float(np.float32(self.scale))


WORKLOADS = {
    "cfg1": Workload("cfg1", 1, FP32, 64, 1000, 1.0, 0, 64,
                     "fp32 64x1000, N(0,1)"),
    "cfg2": Workload("cfg2", 2, BF16, 16384, 2048, 1.0 / math.sqrt(128.0), 1, 512,
                     "bf16 attention scores 16384x2048, N(0,3^2), scale 1/sqrt(128)"),
    "cfg3": Workload("cfg3", 3, BF16, 131072, 128, 1.0, 2, 8192,
                     "bf16 router rows 131072x128, N(0,1) + per-row bias N(0,0.5^2)"),
    "cfg4": Workload("cfg4", 4, BF16, 256, 262144, 1.0, 3, 4,
                     "bf16 vocabulary rows 256x262144, N(0,4^2) + 8 spikes of +30 per row"),
    "cfg5": Workload("cfg5", 5, FP32, 32768, 32768, 1.0, 4, 32,
                     "fp32 causal rows 32768x32768, N(0,2^2), -inf above the diagonal"),
}
N_SPIKES = 8
SPIKE_VALUE = 30.0


def _block(w: Workload, b: int) -> np.ndarray:
    """Rows [b*block_rows, (b+1)*block_rows) of workload w, in stored form."""
    r0 = b * w.block_rows
    nr = min(w.block_rows, w.rows - r0)
    rng = np.random.Generator(np.random.Philox(key=[w.seed, b]))
    if w.index == 1:
        return rng.standard_normal((nr, w.cols), dtype=np.float32)
    if w.index == 2:
        g = rng.standard_normal((nr, w.cols))
        return f64_to_bf16_bits(3.0 * g)
    if w.index == 3:
        g = rng.standard_normal((nr, w.cols))
        bias = 0.5 * rng.standard_normal((nr, 1))
        return f64_to_bf16_bits(g + bias)                 # added in fp64, rounded once
    if w.index == 4:
        g = rng.standard_normal((nr, w.cols))
        x = f64_to_bf16_bits(4.0 * g)
        spike = f64_to_bf16_bits(np.array([SPIKE_VALUE]))[0]
        for r in range(nr):                               # 8 distinct columns per row
            x[r, rng.choice(w.cols, size=N_SPIKES, replace=False)] = spike
        return x
    if w.index == 5:
        x = rng.standard_normal((nr, w.cols), dtype=np.float32)
        x *= np.float32(2.0)                              # exact: N(0, 2^2) on the fp32 grid
        i = np.arange(r0, r0 + nr, dtype=np.int64)[:, None]
        j = np.arange(w.cols, dtype=np.int64)[None, :]
        x[j > i] = -np.inf                                # row i keeps i+1 finite entries
        return x
    raise ValueError(w.name)


def generate_rows(w: Workload, r0: int, r1: int, threads: int = 1) -> np.ndarray:
    """Rows [r0, r1) of workload w as a [r1-r0, cols] array of stored elements."""
    if not (0 <= r0 <= r1 <= w.rows):
        raise ValueError("row range out of bounds")
    out = np.empty((r1 - r0, w.cols), dtype=NP_STORE[w.dtype])
    if r1 == r0:
        return out
    b0, b1 = r0 // w.block_rows, (r1 - 1) // w.block_rows

    def fill(b: int) -> None:
        blk = _block(w, b)
        lo = max(r0, b * w.block_rows)
        hi = min(r1, (b + 1) * w.block_rows)
        out[lo - r0:hi - r0] = blk[lo - b * w.block_rows:hi - b * w.block_rows]

    if threads > 1 and b1 > b0:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(b0, b1 + 1)))
    else:
        for b in range(b0, b1 + 1):
            fill(b)
    return out


def generate(w: Workload, threads: int = 1) -> np.ndarray:
    return generate_rows(w, 0, w.rows, threads=threads)


def checksum(x: np.ndarray) -> int:
    """Order-sensitive 64-bit checksum of the stored bytes (FNV-style over 64-bit words)."""
    raw = np.ascontiguousarray(x).view(np.uint8).ravel()
    pad = (-raw.size) % 8
    if pad:
        raw = np.concatenate([raw, np.zeros(pad, dtype=np.uint8)])
    words = raw.view(np.uint64)
    idx = np.arange(1, words.size + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        mixed = (words ^ (idx * np.uint64(0x9E3779B97F4A7C15))) * np.uint64(0x100000001B3)
        return int(np.bitwise_xor.reduce(mixed) ^ np.uint64(words.size))


class Checksum:
    """The same checksum taken over consecutive slabs of a buffer (rows in order), without holding the buffer:
    `Checksum().update(a).update(b).value() == checksum(np.concatenate([a, b]))` when every slab but the last is
    a whole number of 64-bit words."""

    def __init__(self) -> None:
        self.acc = np.uint64(0)
        self.words = 0

    def update(self, x: np.ndarray, threads: int = 8) -> "Checksum":
        raw = np.ascontiguousarray(x).view(np.uint8).ravel()
        pad = (-raw.size) % 8
        if pad:
            raw = np.concatenate([raw, np.zeros(pad, dtype=np.uint8)])
        words = raw.view(np.uint64)
        step = 1 << 21                                            # bounded temporaries; pieces are independent
        base = self.words

        def piece(i: int) -> np.uint64:
            part = words[i:i + step]
            idx = np.arange(base + i + 1, base + i + part.size + 1, dtype=np.uint64)
            with np.errstate(over="ignore"):
                mixed = (part ^ (idx * np.uint64(0x9E3779B97F4A7C15))) * np.uint64(0x100000001B3)
            return np.bitwise_xor.reduce(mixed)

        starts = range(0, words.size, step)
        if threads > 1 and len(starts) > 1:
            with ThreadPoolExecutor(max_workers=threads) as ex:
                parts = list(ex.map(piece, starts))
        else:
            parts = [piece(i) for i in starts]
        for v in parts:
            self.acc ^= v
        self.words += words.size
        return self

    def value(self) -> int:
        return int(self.acc ^ np.uint64(self.words))


# ---------------------------------------------------------------------------------------------
# generic seeded cases for shape sweeps and special-value rows
# ---------------------------------------------------------------------------------------------

def random_case(rows: int, cols: int, dtype: int, seed: int, sigma: float = 1.0,
                neg_inf_frac: float = 0.0) -> np.ndarray:
    """i.i.d. N(0, sigma^2) rows, optionally with a fraction of entries set to -inf (never a whole row)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, rows * 1_000_003 + cols]))
    g = sigma * rng.standard_normal((rows, cols))
    if neg_inf_frac > 0.0 and cols > 1:
        mask = rng.random((rows, cols)) < neg_inf_frac
        mask[np.arange(rows), rng.integers(0, cols, size=rows)] = False
        g[mask] = -np.inf
    return to_stored(g, dtype)
