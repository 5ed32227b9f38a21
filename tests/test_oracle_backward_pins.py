"""Pins for the oracle's softmax backward: the Jacobian of the softmax taken by 60-digit mpmath
differentiation, PyTorch's float64 autograd, closed forms and invariants. CPU only."""
import mpmath
import numpy as np
import pytest
import torch

from oracle import fso

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16


def mp_softmax(z):
    m = max(z)
    e = [mpmath.exp(v - m) for v in z]
    s = mpmath.fsum(e)
    return [v / s for v in e]


def test_against_the_differentiated_softmax():
    """dx = J^T dy with J_kj = d softmax_k(scale x) / d x_j, each entry by mpmath's numerical derivative."""
    rng = np.random.default_rng(2)
    with mpmath.workdps(60):
        for cols, scale in ((1, 1.0), (2, 0.5), (5, 1.0), (7, -0.75)):
            x = (rng.integers(-12, 12, size=cols) / 4.0).astype(np.float32)
            dy = (rng.integers(-16, 16, size=cols) / 8.0).astype(np.float32)
            sc = float(np.float32(scale))
            y_mp = mp_softmax([mpmath.mpf(sc) * mpmath.mpf(float(v)) for v in x])
            want = []
            for j in range(cols):
                def f(t, j=j):
                    z = [mpmath.mpf(sc) * (t if i == j else mpmath.mpf(float(x[i]))) for i in range(cols)]
                    p = mp_softmax(z)
                    return mpmath.fsum(mpmath.mpf(float(dy[k])) * p[k] for k in range(cols))
                want.append(float(mpmath.diff(f, mpmath.mpf(float(x[j])))))
            # the oracle takes y as a stored tensor: give it the exact softmax rounded to fp32 and allow for that rounding
            y32 = np.array([float(v) for v in y_mp], dtype=np.float32)
            got = fso.softmax_backward_f64(dy[None, :], y32[None, :], FP32, scale)[0]
            assert np.max(np.abs(got - np.array(want))) < 5e-7 * max(1.0, float(np.max(np.abs(dy)))) * abs(sc) + 1e-12


@pytest.mark.parametrize("dtype,tdt", [(FP32, torch.float32), (BF16, torch.bfloat16), (FP16, torch.float16)])
def test_against_torch_softmax_backward_float64(dtype, tdt):
    g = torch.Generator().manual_seed(9 + dtype)
    for rows, cols in ((2, 5), (3, 1000), (1, 4097)):
        y = torch.softmax(torch.randn(rows, cols, generator=g) * 2, -1).to(tdt)
        dy = torch.randn(rows, cols, generator=g).to(tdt)
        for scale in (1.0, 0.25):
            sc = float(np.float32(scale))
            want = (torch.ops.aten._softmax_backward_data(dy.double(), y.double(), -1, torch.float64) * sc).numpy()
            bits = (lambda t: t.numpy()) if dtype == FP32 else (lambda t: t.view(torch.int16).numpy().view(np.uint16))
            got = fso.softmax_backward_f64(bits(dy), bits(y), dtype, scale)
            assert np.max(np.abs(got - want)) < 1e-13 * max(1.0, float(np.max(np.abs(want))))


def test_closed_forms_and_invariants():
    y = np.array([[0.5, 0.25, 0.125, 0.125]], dtype=np.float32)
    # a constant upstream gradient gives zero (the softmax ignores shifts): exact, the products are exact in fp64
    dx = fso.softmax_backward_f64(np.full((1, 4), 3.0, np.float32), y, FP32, 1.0)
    assert np.array_equal(dx, np.zeros((1, 4)))
    # a one-hot gradient at i: dx_j = scale * y_j * (delta_ij - y_i)
    dy = np.array([[0.0, 1.0, 0.0, 0.0]], dtype=np.float32)
    dx = fso.softmax_backward_f64(dy, y, FP32, 2.0)
    assert np.array_equal(dx, 2.0 * y.astype(np.float64) * (dy - 0.25))
    # the gradient sums to zero along the row when y sums to one
    rng = np.random.default_rng(1)
    dy = rng.standard_normal((3, 4)).astype(np.float32)
    dx = fso.softmax_backward_f64(dy, np.repeat(y, 3, 0), FP32, 0.5)
    assert np.max(np.abs(dx.sum(axis=1))) < 1e-15
    # special values follow IEEE: a NaN in dy poisons its row, a zero y gives a zero gradient there
    dyn = dy.copy(); dyn[1, 2] = np.nan
    dx = fso.softmax_backward_f64(dyn, np.repeat(y, 3, 0), FP32, 1.0)
    assert np.all(np.isnan(dx[1])) and not np.any(np.isnan(dx[0])) and not np.any(np.isnan(dx[2]))
    y0 = np.array([[1.0, 0.0]], dtype=np.float32)
    assert np.array_equal(fso.softmax_backward_f64(np.array([[2.0, 5.0]], np.float32), y0, FP32, 1.0), [[0.0, 0.0]])
