"""fp64 oracle of the row normalisations -- TEST INFRASTRUCTURE, not the product.

layer_norm and group_norm are the two normalisation operators the paper reports generated kernels
for (Sec. IV-C, Stable Diffusion 3.5 Medium: group normalization 1.699x, layer normalization
1.049x over eager). The paper gives no formula; these are the operators' public definitions:

    layer_norm   y_ij = (x_ij - mu_i) / sqrt(var_i + eps) * gamma_j + beta_j
                 mu_i = mean_j x_ij,  var_i = mean_j (x_ij - mu_i)^2          (biased variance)
    group_norm   x: [n, channels, spatial]; each (sample, group) of channels/groups * spatial
                 contiguous elements is normalised like one row; gamma, beta are per channel.

Written out in numpy float64, one step per line, no blocking or fusion. Stored 16-bit inputs are
widened exactly with the softmax oracle's decoders (pinned exhaustively by its own tests).

Only tests, the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs may
import this module. It never touches CUDA and shares nothing with the CUDA library.

Pins (tests/test_oracle_norm_pins.py): 50-digit mpmath values stored under tests/golden/, PyTorch's
float64 CPU operators as an independent library, closed forms (constant rows, two-element rows),
invariants (zero mean, sum of squares, shift and scale invariance), and a pure-Python loop over a
tiny group_norm tensor for the channel indexing; the two error scales that set binary32 tolerances
(error_scale, backward_error_scale) by hand-computed rows and by bracketing a binary32 evaluation
against 60-digit arithmetic. Nothing here is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import fso

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16


def _widen_opt(a, dtype):
    return None if a is None else fso.widen(np.ascontiguousarray(a), dtype)


def layer_norm_f64(x: np.ndarray, dtype: int, gamma=None, beta=None, eps: float = 1e-5) -> np.ndarray:
    """x: [rows, cols] stored elements; gamma, beta: [cols] stored elements or None. Returns float64."""
    X = fso.widen(np.ascontiguousarray(x), dtype)
    if X.ndim != 2:
        raise ValueError("x must be [rows, cols]")
    rows, cols = X.shape
    g = _widen_opt(gamma, dtype)
    b = _widen_opt(beta, dtype)
    e = float(np.float32(eps))                      # eps crosses the C ABI as a float
    with np.errstate(all="ignore"):
        mu = X.sum(axis=1, keepdims=True) / cols
        d = X - mu
        var = (d * d).sum(axis=1, keepdims=True) / cols
        y = d / np.sqrt(var + e)
        if g is not None:
            y = y * g[None, :]
        if b is not None:
            y = y + b[None, :]
    return y


def group_norm_f64(x: np.ndarray, dtype: int, groups: int, gamma=None, beta=None, eps: float = 1e-5) -> np.ndarray:
    """x: [n, channels, spatial] stored elements; gamma, beta: [channels] or None. Returns float64."""
    X = fso.widen(np.ascontiguousarray(x), dtype)
    if X.ndim != 3:
        raise ValueError("x must be [n, channels, spatial]")
    n, ch, sp = X.shape
    if groups < 1 or ch % groups:
        raise ValueError("channels must be a multiple of groups")
    g = _widen_opt(gamma, dtype)
    b = _widen_opt(beta, dtype)
    e = float(np.float32(eps))
    cpg = ch // groups
    m = cpg * sp
    with np.errstate(all="ignore"):
        G = X.reshape(n, groups, m)
        mu = G.sum(axis=2, keepdims=True) / m
        d = G - mu
        var = (d * d).sum(axis=2, keepdims=True) / m
        y = (d / np.sqrt(var + e)).reshape(n, ch, sp)
        if g is not None:
            y = y * g[None, :, None]
        if b is not None:
            y = y + b[None, :, None]
    return y


def error_scale(x: np.ndarray, dtype: int, rows_shape, gamma_full=None, beta_full=None, eps: float = 1e-5) -> np.ndarray:
    """Per-element magnitude that a binary32 evaluation's rounding error is proportional to:
    |gamma| * (|x - mu| + mean|x|) / sqrt(var + eps) + |beta|, for x viewed as `rows_shape`
    ([rows, cols]); gamma_full / beta_full are float64 arrays broadcastable to that shape.
    The first term carries the errors of mu (proportional to mean|x|), of x - mu and of the
    reciprocal standard deviation; the second the final addition."""
    X = fso.widen(np.ascontiguousarray(x), dtype).reshape(rows_shape)
    cols = X.shape[1]
    e = float(np.float32(eps))
    with np.errstate(all="ignore"):
        mu = X.sum(axis=1, keepdims=True) / cols
        d = X - mu
        var = (d * d).sum(axis=1, keepdims=True) / cols
        s = (np.abs(d) + np.abs(X).sum(axis=1, keepdims=True) / cols) / np.sqrt(var + e)
        if gamma_full is not None:
            s = s * np.abs(gamma_full)
        if beta_full is not None:
            s = s + np.abs(beta_full)
    return s


def backward_error_scale(dy: np.ndarray, y: np.ndarray, dtype: int, scale: float) -> np.ndarray:
    """Per-element magnitude that the rounding error of a binary32 evaluation of the softmax gradient
    dx = scale * y * (dy - sum_k dy_k y_k) is proportional to: |scale| |y| (|dy| + sum_k |dy_k y_k|). dy and the dot
    product can cancel, so the error is not proportional to |dx|; the second term carries the rounding of the
    binary32 products and of their sum. dy, y: [rows, cols] stored elements."""
    g = fso.widen(np.ascontiguousarray(dy), dtype)
    p = fso.widen(np.ascontiguousarray(y), dtype)
    sc = abs(float(np.float32(scale)))
    with np.errstate(all="ignore"):
        return sc * np.abs(p) * (np.abs(g) + np.abs(g * p).sum(axis=1, keepdims=True))


def log_softmax_bound(want: np.ndarray) -> np.ndarray:
    """Absolute fp32 bound of a log_softmax output: 1e-6 * max(1, |y|) -- three binary32 roundings of
    (x - R) * scale - ln S plus 2^-22 absolute on log2 S; relative above 1 because outputs reach -50 and beyond.
    Non-finite oracle values (a -inf output, a NaN row) get 1e-6: they are compared exactly elsewhere."""
    w = np.asarray(want, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        return 1e-6 * np.maximum(1.0, np.where(np.isfinite(w), np.abs(w), 1.0))


def masked_softmax_bound(x: np.ndarray, mask: np.ndarray, dtype: int, q_rows: int, heads: int, scale: float,
                         want: np.ndarray) -> np.ndarray:
    """Absolute fp32 bound of softmax(scale * x + mask): 1e-6 + 2.5e-7 * Z * y, Z the largest finite |scale * x + mask|
    of the row. The exponent scale * x + mask is formed in binary32 before the row maximum is taken off, so it
    carries a rounding of relative size 2^-24 of a number as large as Z: 2^-24 * Z * ln 2 on the exponent of the element
    and as much again through the row sum. x: [rows, cols] ordered (batch, head, query), mask: [rows / heads, cols]."""
    X = fso.widen(np.ascontiguousarray(x), dtype)
    M = fso.widen(np.ascontiguousarray(mask), dtype)
    rows = X.shape[0]
    mrow = (np.arange(rows) // (heads * q_rows)) * q_rows + np.arange(rows) % q_rows
    sc = float(np.float32(scale))
    w = np.asarray(want, dtype=np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        z = sc * X + M[mrow]
        zmax = np.max(np.where(np.isfinite(z), np.abs(z), 0.0), axis=1, keepdims=True)
        return 1e-6 + 2.5e-7 * zmax * np.where(np.isfinite(w), w, 1.0)


@dataclass
class NormReport:
    max_rel_err: float      # max over elements of |got - want| / error_scale
    max_ulp: int            # 16-bit: max distance to the correctly rounded value among elements outside the fp32 bound
    nan_mismatch: int
    n_compared: int
    worst_index: int

    def ok(self, dtype: int, rel_tol: float = 2e-6, ulp_tol: int = 1) -> bool:
        if self.nan_mismatch:
            return False
        return self.max_rel_err <= rel_tol if dtype == FP32 else self.max_ulp <= ulp_tol


def compare(got: np.ndarray, dtype: int, want: np.ndarray, scale: np.ndarray, rel_tol: float = 2e-6) -> NormReport:
    """fp32: |got - want| / scale (reported as max_rel_err; the bar is rel_tol).
    16-bit: an element passes when it is within one unit in the last place of the fp64 value
    rounded once to the format, or within rel_tol * scale of the fp64 value (where gamma * n and
    beta cancel, the fp32 evaluation's error can exceed the spacing of the small result);
    max_ulp reports the worst element that needed the first rule."""
    want = np.ascontiguousarray(want, dtype=np.float64).ravel()
    scale = np.ascontiguousarray(np.broadcast_to(scale, np.shape(got)), dtype=np.float64).ravel()
    g64 = fso.widen(np.ascontiguousarray(got), dtype).ravel()
    gn, wn = np.isnan(g64), np.isnan(want)
    nan_mismatch = int(np.count_nonzero(gn != wn))
    live = ~(gn | wn)
    with np.errstate(all="ignore"):
        err = np.abs(g64 - want)
        same_inf = np.isinf(want) & (g64 == want)
        err = np.where(same_inf, 0.0, err)
        rel = np.where(live, err / np.maximum(scale, 1e-300), 0.0)
        rel = np.where(live & (err == 0.0), 0.0, rel)
    max_ulp = 0
    worst = int(np.argmax(rel)) if rel.size else -1
    if dtype != FP32 and rel.size:
        wr = fso.round_from_f64(want, dtype).astype(np.int32)
        gb = np.ascontiguousarray(got).view(np.uint16).ravel().astype(np.int32)

        def ordinal(b):
            return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)

        ulp = np.abs(ordinal(gb) - ordinal(wr))
        need = live & ~(rel <= rel_tol)
        if np.any(need):
            max_ulp = int(ulp[need].max())
            worst = int(np.argmax(np.where(need, ulp, -1)))
    return NormReport(float(rel.max()) if rel.size else 0.0, max_ulp, nan_mismatch, int(np.count_nonzero(live)), worst)
