"""Pins for the oracle's log_softmax: 100-digit mpmath on small rows, PyTorch's float64 CPU operator,
closed forms and invariants -- never the oracle's own output. CPU only."""
import math

import mpmath
import numpy as np
import pytest
import torch

from oracle import fso
from paper_2607_24762_b200 import workloads as W

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16


def mp_log_softmax(row, scale):
    with mpmath.workdps(100):
        z = [mpmath.mpf(float(scale)) * mpmath.mpf(float(v)) for v in row]
        m = max(z)
        s = mpmath.fsum(mpmath.exp(v - m) for v in z)
        return [float(v - m - mpmath.log(s)) for v in z]


def test_small_rows_vs_mpmath():
    rng = np.random.default_rng(4)
    for cols in (1, 2, 3, 7, 16, 33):
        for scale in (1.0, 0.5, -1.0, 0.0, float(np.float32(128 ** -0.5))):
            x = (rng.integers(-200, 200, size=(3, cols)) / 8.0).astype(np.float32)
            y = fso.log_softmax_f64(x, FP32, scale)
            for i in range(3):
                want = np.array(mp_log_softmax(x[i], float(np.float32(scale))))
                assert np.max(np.abs(y[i] - want) / np.maximum(1.0, np.abs(want))) < 1e-14


@pytest.mark.parametrize("dtype,tdt", [(FP32, torch.float32), (BF16, torch.bfloat16), (FP16, torch.float16)])
def test_against_torch_float64(dtype, tdt):
    g = torch.Generator().manual_seed(3 + dtype)
    for rows, cols in ((2, 5), (3, 1000), (1, 4097)):
        xt = (torch.randn(rows, cols, generator=g) * 4).to(tdt)
        xs = xt.numpy() if dtype == FP32 else xt.view(torch.int16).numpy().view(np.uint16)
        for scale in (1.0, 0.25):
            want = torch.log_softmax(xt.double() * float(np.float32(scale)), dim=-1).numpy()
            got = fso.log_softmax_f64(xs, dtype, scale)
            assert np.max(np.abs(got - want)) < 1e-12 * max(1.0, float(np.max(np.abs(want))))


def test_closed_forms_and_invariants():
    # a uniform row: y = -ln n, whatever the value and the scale
    for n in (1, 2, 10, 4096):
        y = fso.log_softmax_f64(np.full((1, n), 2.5, dtype=np.float32), FP32, 0.75)
        assert np.max(np.abs(y + math.log(n))) < 1e-15 * max(1.0, math.log(n) if n > 1 else 1.0) + 1e-15
    # two elements a, b: y = -ln(1 + exp(-(a-b))) for the larger one
    y = fso.log_softmax_f64(np.array([[3.0, 1.0]], dtype=np.float32), FP32, 1.0)
    assert abs(y[0, 0] + math.log1p(math.exp(-2.0))) < 1e-15 and abs(y[0, 1] + 2.0 + math.log1p(math.exp(-2.0))) < 1e-15
    # exp(log_softmax) is the (separately pinned) softmax; logsumexp of the result is 0; shifts cancel
    x = W.random_case(5, 300, FP32, seed=8, sigma=3.0, neg_inf_frac=0.05)
    x = (np.round(x * 16) / 16).astype(np.float32)          # on a grid, so that the shift below is exact
    y = fso.log_softmax_f64(x, FP32, 0.5)
    p = fso.softmax_f64(x, FP32, 0.5)
    assert np.max(np.abs(np.exp(y) - p)) < 1e-15
    assert np.max(np.abs(np.log(np.exp(y).sum(axis=1)))) < 1e-14
    finite = np.isfinite(x)
    xs = np.where(finite, x + np.float32(8.0), x).astype(np.float32)                  # exact shifts of the finite entries
    ys = fso.log_softmax_f64(xs, FP32, 0.5)
    assert np.max(np.abs(np.where(finite, ys - y, 0.0))) < 1e-13
    assert np.all(np.isneginf(y[~finite])) and np.all(y[finite] <= 0.0)


def test_special_values():
    inf = np.inf
    x = np.array([[1.0, -inf, 2.0], [1.0, np.nan, 2.0], [1.0, inf, 2.0], [-inf, -inf, -inf]], dtype=np.float32)
    y = fso.log_softmax_f64(x, FP32, 1.0)
    assert np.isneginf(y[0, 1]) and np.isfinite(y[0, 0]) and np.isfinite(y[0, 2])
    assert np.all(np.isnan(y[1])) and np.all(np.isnan(y[2])) and np.all(np.isnan(y[3]))
    # a negative scale turns the smallest x into the reference
    y = fso.log_softmax_f64(np.array([[1.0, 2.0, 3.0]], dtype=np.float32), FP32, -1.0)
    want = mp_log_softmax([1.0, 2.0, 3.0], -1.0)
    assert np.max(np.abs(y[0] - np.array(want))) < 1e-15
    assert fso.log_softmax_f64(np.zeros((0, 4), np.float32), FP32).shape == (0, 4)


def test_log_softmax_bound_values_and_bracket():
    """1e-6 * max(1, |y|): by hand, and against a binary32 evaluation of y = (x - R) * scale - ln S (numpy float32, three
    summation orders) measured with 60-digit arithmetic: its worst error is between 3 % and 100 % of the bound on rows
    whose outputs are of order one and on rows whose outputs reach the hundreds. Ten times looser fails."""
    import mpmath as mp
    from oracle import fno
    b = fno.log_softmax_bound(np.array([0.0, -0.5, -1.0, -50.0, -np.inf, np.nan, 300.0]))
    assert np.allclose(b, [1e-6, 1e-6, 1e-6, 5e-5, 1e-6, 1e-6, 3e-4], rtol=1e-14, atol=0)
    rng = np.random.default_rng(31)
    with mp.workdps(60):
        for rows, cols, sigma, scale in ((4, 257, 1.0, 1.0), (3, 64, 4.0, 0.5), (3, 1000, 30.0, 1.0), (3, 96, 100.0, -2.0)):
            x = (rng.standard_normal((rows, cols)) * sigma).astype(np.float32)
            want = fso.log_softmax_f64(x, FP32, scale)
            bound = fno.log_softmax_bound(want)
            sc = np.float32(scale)
            z = x if scale > 0 else -x
            r = z.max(axis=1, keepdims=True)
            d = ((z - r).astype(np.float32) * np.abs(sc)).astype(np.float32)
            e = np.exp(d).astype(np.float32)
            worst = 0.0
            for order in (np.arange(cols), np.arange(cols)[::-1], np.random.default_rng(cols).permutation(cols)):
                ssum = np.zeros(rows, dtype=np.float32)
                for j in order:
                    ssum = (ssum + e[:, j]).astype(np.float32)
                got = (d - np.log(ssum).astype(np.float32)[:, None]).astype(np.float32)
                worst = max(worst, float(np.max(np.abs(got.astype(np.float64) - want) / bound)))
            assert 0.03 <= worst <= 1.0, (rows, cols, sigma, scale, worst)
