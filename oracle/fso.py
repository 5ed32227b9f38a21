"""ctypes front end of the fp64 softmax oracle -- TEST INFRASTRUCTURE, not the product.

Only tests, the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs may
import this module. It never touches CUDA and shares nothing with the CUDA library; inputs come
in as numpy arrays of the stored bit patterns (float32, or uint16 for bf16/fp16).

The arithmetic lives in ``fso_oracle.cpp`` (g++, ``-ffp-contract=off``, no fast-math); this file
only builds it on first use and marshals arguments.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

FP32, BF16, FP16 = 0, 1, 2
_ESIZE = {FP32: 4, BF16: 2, FP16: 2}
_NP_STORE = {FP32: np.float32, BF16: np.uint16, FP16: np.uint16}

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fso_oracle.cpp")
_LIB = os.path.join(_HERE, "libfso_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (host only). Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-o", _LIB + ".tmp", _SRC]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


class _Report(ctypes.Structure):
    _fields_ = [("max_abs_err", ctypes.c_double), ("max_ulp", ctypes.c_int64),
                ("nan_mismatch", ctypes.c_int64), ("zero_mismatch", ctypes.c_int64),
                ("negative", ctypes.c_int64), ("worst_index", ctypes.c_int64),
                ("n_compared", ctypes.c_int64)]


@dataclass
class Report:
    max_abs_err: float
    max_ulp: int
    nan_mismatch: int
    zero_mismatch: int
    negative: int
    worst_index: int
    n_compared: int

    def ok(self, dtype: int, abs_tol: float = 1e-6, ulp_tol: int = 1) -> bool:
        """The stated bar: fp32 max |delta| <= 1e-6; 16-bit within 1 ulp of the rounded fp64 value."""
        if self.nan_mismatch or self.zero_mismatch or self.negative:
            return False
        return self.max_abs_err <= abs_tol if dtype == FP32 else self.max_ulp <= ulp_tol


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            vp, i64, f32, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_int
            lib.fso_softmax_f64.argtypes = [vp, ci, i64, i64, f32, vp]
            lib.fso_softmax_f64.restype = None
            lib.fso_softmax_row_f64.argtypes = [vp, ci, i64, f32, vp]
            lib.fso_softmax_row_f64.restype = None
            lib.fso_log_softmax_f64.argtypes = [vp, ci, i64, i64, f32, vp]
            lib.fso_log_softmax_f64.restype = None
            lib.fso_softmax_backward_f64.argtypes = [vp, vp, ci, i64, i64, f32, vp]
            lib.fso_softmax_backward_f64.restype = None
            lib.fso_softmax_masked_f64.argtypes = [vp, vp, ci, i64, i64, i64, i64, f32, vp]
            lib.fso_softmax_masked_f64.restype = None
            lib.fso_softmax_causal_f64.argtypes = [vp, ci, i64, i64, i64, f32, vp]
            lib.fso_softmax_causal_f64.restype = None
            lib.fso_router_topk_f64.argtypes = [vp, ci, i64, i64, i64, f32, ci, vp, vp]
            lib.fso_router_topk_f64.restype = None
            lib.fso_widen.argtypes = [vp, ci, i64, vp]
            lib.fso_widen.restype = None
            lib.fso_round_from_f64.argtypes = [vp, ci, i64, vp]
            lib.fso_round_from_f64.restype = None
            lib.fso_compare.argtypes = [vp, ci, vp, i64, ctypes.POINTER(_Report)]
            lib.fso_compare.restype = None
            _lib = lib
    return _lib


def _stored(x: np.ndarray, dtype: int) -> np.ndarray:
    want = _NP_STORE[dtype]
    if dtype == FP16 and x.dtype == np.float16:
        x = x.view(np.uint16)
    if x.dtype != want:
        raise TypeError(f"dtype {dtype} expects a {np.dtype(want)} array of stored bits, got {x.dtype}")
    return np.ascontiguousarray(x)


def softmax_f64(x: np.ndarray, dtype: int, scale: float = 1.0) -> np.ndarray:
    """fp64 softmax over the last axis of a 2-D array of stored elements."""
    x = _stored(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, cols]")
    rows, cols = x.shape
    y = np.empty((rows, cols), dtype=np.float64)
    if rows and cols:
        _load().fso_softmax_f64(x.ctypes.data, dtype, rows, cols, np.float32(scale), y.ctypes.data)
    return y


def log_softmax_f64(x: np.ndarray, dtype: int, scale: float = 1.0) -> np.ndarray:
    """fp64 log_softmax over the last axis of a 2-D array of stored elements."""
    x = _stored(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, cols]")
    rows, cols = x.shape
    y = np.empty((rows, cols), dtype=np.float64)
    if rows and cols:
        _load().fso_log_softmax_f64(x.ctypes.data, dtype, rows, cols, np.float32(scale), y.ctypes.data)
    return y


def softmax_backward_f64(dy: np.ndarray, y: np.ndarray, dtype: int, scale: float = 1.0) -> np.ndarray:
    """fp64 gradient of softmax(scale * x) with respect to x, from the upstream gradient dy and the output y."""
    dy, y = _stored(dy, dtype), _stored(y, dtype)
    if dy.ndim != 2 or dy.shape != y.shape:
        raise ValueError("dy and y must be [rows, cols] of the same shape")
    rows, cols = y.shape
    dx = np.empty((rows, cols), dtype=np.float64)
    if rows and cols:
        _load().fso_softmax_backward_f64(dy.ctypes.data, y.ctypes.data, dtype, rows, cols, np.float32(scale), dx.ctypes.data)
    return dx


def softmax_masked_f64(x: np.ndarray, mask: np.ndarray, dtype: int, q_rows: int, heads: int, scale: float = 1.0) -> np.ndarray:
    """fp64 softmax(scale * x + mask): x [rows, cols] ordered (batch, head, query), mask [batch * q_rows, cols]."""
    x, mask = _stored(x, dtype), _stored(mask, dtype)
    rows, cols = x.shape
    if q_rows < 1 or heads < 1 or rows % (q_rows * heads) or mask.shape != (rows // heads, cols):
        raise ValueError("rows must be batch * heads * q_rows and mask [batch * q_rows, cols]")
    y = np.empty((rows, cols), dtype=np.float64)
    if rows and cols:
        _load().fso_softmax_masked_f64(x.ctypes.data, mask.ctypes.data, dtype, rows, cols, q_rows, heads, np.float32(scale),
                                       y.ctypes.data)
    return y


def softmax_causal_f64(x: np.ndarray, dtype: int, q_offset: int, scale: float = 1.0) -> np.ndarray:
    """fp64 causal softmax: row i keeps columns j <= i + q_offset; masked columns give exactly 0."""
    x = _stored(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, cols]")
    rows, cols = x.shape
    y = np.empty((rows, cols), dtype=np.float64)
    if rows and cols:
        _load().fso_softmax_causal_f64(x.ctypes.data, dtype, rows, cols, q_offset, np.float32(scale), y.ctypes.data)
    return y


def router_topk_f64(x: np.ndarray, dtype: int, k: int, scale: float = 1.0, renorm: bool = False):
    """fp64 router step: (weights [rows, k] float64, indices [rows, k] int32), largest first."""
    x = _stored(x, dtype)
    rows, cols = x.shape
    if not (1 <= k <= cols):
        raise ValueError("k out of range")
    w = np.empty((rows, k), dtype=np.float64)
    idx = np.empty((rows, k), dtype=np.int32)
    if rows:
        _load().fso_router_topk_f64(x.ctypes.data, dtype, rows, cols, k, np.float32(scale), int(renorm),
                                    w.ctypes.data, idx.ctypes.data)
    return w, idx


def widen(x: np.ndarray, dtype: int) -> np.ndarray:
    x = _stored(x, dtype)
    out = np.empty(x.shape, dtype=np.float64)
    _load().fso_widen(x.ctypes.data, dtype, x.size, out.ctypes.data)
    return out


def round_from_f64(v: np.ndarray, dtype: int) -> np.ndarray:
    """Round-to-nearest-even of fp64 values to the stored format (bit patterns for 16-bit)."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=_NP_STORE[dtype])
    _load().fso_round_from_f64(v.ctypes.data, dtype, v.size, out.ctypes.data)
    return out


def compare(got: np.ndarray, dtype: int, want: np.ndarray) -> Report:
    """Apply the parity rule to a result in its stored dtype against fp64 oracle values."""
    got = _stored(got, dtype)
    want = np.ascontiguousarray(want, dtype=np.float64)
    if got.size != want.size:
        raise ValueError("size mismatch")
    rep = _Report()
    _load().fso_compare(got.ctypes.data, dtype, want.ctypes.data, got.size, ctypes.byref(rep))
    return Report(rep.max_abs_err, rep.max_ulp, rep.nan_mismatch, rep.zero_mismatch, rep.negative,
                  rep.worst_index, rep.n_compared)
