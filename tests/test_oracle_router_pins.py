"""Pins for the oracle's router step (softmax over experts, then top-k, optional renormalisation):
expected values from mpmath + Python's own sort, closed forms and invariants. CPU only."""
import mpmath
import numpy as np
import pytest

from oracle import fso
from paper_2607_24762_b200 import workloads as W

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16


def mp_router(row, k, scale, renorm):
    with mpmath.workdps(80):
        z = [mpmath.mpf(float(scale)) * mpmath.mpf(float(v)) for v in row]
        m = max(z)
        e = [mpmath.exp(v - m) for v in z]
        s = mpmath.fsum(e)
        order = sorted(range(len(row)), key=lambda j: (-z[j], j))[:k]
        sel = mpmath.fsum(e[j] for j in order)
        w = [float(e[j] / (sel if renorm else s)) for j in order]
    return w, order


@pytest.mark.parametrize("renorm", [False, True])
def test_small_rows_vs_mpmath_and_python_sort(renorm):
    rng = np.random.default_rng(12)
    for cols in (1, 2, 5, 8, 16):
        x = (rng.integers(-12, 12, size=(6, cols)) / 2.0).astype(np.float32)      # many ties
        for k in sorted({1, min(2, cols), cols}):
            for scale in (1.0, 0.3, -1.0, 0.0):
                w, idx = fso.router_topk_f64(x, FP32, k, scale, renorm)
                for i in range(6):
                    ww, oo = mp_router(x[i], k, float(np.float32(scale)), renorm)
                    assert list(idx[i]) == oo, (cols, k, scale, i)
                    assert np.allclose(w[i], ww, rtol=1e-14, atol=0)


def test_full_k_is_the_sorted_softmax_and_k1_is_argmax():
    x = W.random_case(5, 64, BF16, seed=2, sigma=2.0)
    y = fso.softmax_f64(x, BF16, 0.5)
    w, idx = fso.router_topk_f64(x, BF16, 64, 0.5)
    for i in range(5):
        assert sorted(idx[i]) == list(range(64))
        assert np.array_equal(w[i], y[i, idx[i]]) and np.all(np.diff(w[i]) <= 0)
    w1, i1 = fso.router_topk_f64(x, BF16, 1, 0.5)
    xf = W.stored_to_f32(x, BF16)
    assert np.array_equal(i1[:, 0], np.argmax(xf, axis=1))      # numpy's argmax also takes the first maximum
    wr, ir = fso.router_topk_f64(x, BF16, 8, 0.5, renorm=True)
    assert np.allclose(wr.sum(axis=1), 1.0, atol=1e-15) and np.array_equal(ir, idx[:, :8])
    assert np.allclose(wr, w[:, :8] / w[:, :8].sum(axis=1, keepdims=True), rtol=1e-15)


def test_ties_go_to_the_lower_column_and_special_values():
    x = np.array([[1.0, 3.0, 3.0, 0.0, 3.0, -np.inf],
                  [np.nan, 1.0, 2.0, 0.0, 0.0, 0.0],
                  [-np.inf] * 6], dtype=np.float32)
    w, idx = fso.router_topk_f64(x, FP32, 4, 1.0)
    assert list(idx[0]) == [1, 2, 4, 0]
    assert np.all(np.isnan(w[1])) and list(idx[1]) == [2, 1, 3, 4]          # NaN counts as the smallest key
    assert np.all(np.isnan(w[2])) and list(idx[2]) == [0, 1, 2, 3]
    w, idx = fso.router_topk_f64(x[:1], FP32, 3, -1.0)                      # negative scale: smallest x first
    assert np.all(np.isnan(w)) and list(idx[0])[0] == 5                      # -1 * -inf = +inf wins and poisons p
