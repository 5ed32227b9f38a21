"""Pins for the oracle's causal softmax (row i keeps columns j <= i + q_offset): expected values come
from 100-digit mpmath on the kept prefix, closed forms and invariants, not from the oracle. CPU only."""
import itertools

import mpmath
import numpy as np
import pytest

from oracle import fso
from paper_2607_24762_b200 import workloads as W

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16


def mp_prefix_softmax(row, keep, scale):
    out = [0.0] * len(row)
    if keep == 0:
        return [float("nan")] * len(row)
    with mpmath.workdps(100):
        z = [mpmath.mpf(float(scale)) * mpmath.mpf(float(v)) for v in row[:keep]]
        m = max(z)
        e = [mpmath.exp(v - m) for v in z]
        s = mpmath.fsum(e)
        for j, v in enumerate(e):
            out[j] = float(v / s)
    return out


@pytest.mark.parametrize("q_offset", [-2, -1, 0, 1, 3, 10])
def test_bruteforce_small_matrices_vs_mpmath(q_offset):
    rng = np.random.default_rng(7 + q_offset)
    for rows, cols in ((1, 1), (4, 4), (3, 6), (6, 3), (5, 9)):
        x = (rng.integers(-24, 24, size=(rows, cols)) / 4.0).astype(np.float32)
        for scale in (1.0, 0.5, -1.0, 0.0):
            y = fso.softmax_causal_f64(x, FP32, q_offset, scale)
            for i in range(rows):
                keep = min(cols, max(0, i + q_offset + 1))
                want = np.array(mp_prefix_softmax(x[i], keep, float(np.float32(scale))))
                if keep == 0:
                    assert np.all(np.isnan(y[i]))
                    continue
                assert np.all(y[i, keep:] == 0.0) and not np.any(np.signbit(y[i, keep:]))
                ulp = np.abs(y[i, :keep].view(np.int64) - want[:keep].view(np.int64))
                assert ulp.max() <= 2, (rows, cols, i, scale)


def test_masked_inputs_are_never_looked_at():
    x = W.random_case(6, 11, FP32, seed=3, sigma=2.0)
    a = fso.softmax_causal_f64(x, FP32, 2, 1.0)
    poisoned = x.copy()
    for i in range(6):
        poisoned[i, i + 3:] = [np.nan, np.inf, -np.inf, 1e30, -1e30, 0.0, 5.0, np.nan][: max(0, 11 - i - 3)]
    b = fso.softmax_causal_f64(poisoned, FP32, 2, 1.0)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_no_mask_left_equals_plain_softmax_and_square_case(dtype):
    x = W.random_case(5, 8, dtype, seed=9, sigma=1.5)
    assert np.array_equal(fso.softmax_causal_f64(x, dtype, 7, 0.7), fso.softmax_f64(x, dtype, 0.7))
    assert np.array_equal(fso.softmax_causal_f64(x, dtype, 100, 0.7), fso.softmax_f64(x, dtype, 0.7))
    y = fso.softmax_causal_f64(x, dtype, 0, 1.0)
    assert y[0, 0] == 1.0 and np.all(y[0, 1:] == 0.0)
    for i in range(5):
        assert np.count_nonzero(y[i]) == i + 1 and abs(y[i].sum() - 1.0) < 1e-15
        sub = fso.softmax_f64(np.ascontiguousarray(x[i:i + 1, :i + 1]), dtype, 1.0)
        assert np.array_equal(y[i, :i + 1], sub[0])              # the kept prefix is a plain softmax


def test_equals_plain_softmax_of_an_explicitly_masked_input():
    w = W.WORKLOADS["cfg5"]
    x = W.generate_rows(w, 0, 40)[:, :64].copy()                 # rows 0..39 of the causal workload, 64 columns
    x[~np.isfinite(x)] = 3.0                                     # drop the workload's own -inf mask
    masked = x.copy()
    for i in range(40):
        masked[i, i + 1:] = -np.inf
    assert np.array_equal(fso.softmax_causal_f64(x, FP32, 0, 1.0), fso.softmax_f64(masked, FP32, 1.0))


def test_rows_without_any_kept_column_are_nan():
    x = np.zeros((4, 5), dtype=np.float32)
    y = fso.softmax_causal_f64(x, FP32, -2, 1.0)
    assert np.all(np.isnan(y[0])) and np.all(np.isnan(y[1]))
    assert np.array_equal(y[2], [1, 0, 0, 0, 0]) and np.array_equal(y[3], [0.5, 0.5, 0, 0, 0])
