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


# ---------------------------------------------------------------------------------------------
# backward_error_scale: the magnitude the binary32 tolerance of the backward's parity tests multiplies
# ---------------------------------------------------------------------------------------------

def test_backward_error_scale_hand_computed():
    """|scale| |y| (|dy| + sum |dy y|) worked out by hand: y = [1/4, 3/4], dy = [2, -4]: sum |dy y| = 1/2 + 3 = 7/2."""
    from oracle import fno
    y = np.array([[0.25, 0.75]], dtype=np.float32)
    dy = np.array([[2.0, -4.0]], dtype=np.float32)
    assert np.array_equal(fno.backward_error_scale(dy, y, FP32, 1.0), [[0.25 * 5.5, 0.75 * 7.5]])
    assert np.array_equal(fno.backward_error_scale(dy, y, FP32, -0.5), [[0.125 * 5.5, 0.375 * 7.5]])
    # rows are independent, and a one-hot y silences every other column
    y2 = np.array([[0.25, 0.75], [1.0, 0.0]], dtype=np.float32)
    dy2 = np.array([[2.0, -4.0], [3.0, 100.0]], dtype=np.float32)
    assert np.array_equal(fno.backward_error_scale(dy2, y2, FP32, 1.0), [[0.25 * 5.5, 0.75 * 7.5], [6.0, 0.0]])


def test_backward_error_scale_brackets_a_binary32_evaluation():
    """A binary32 evaluation of the gradient, one rounding per operation and three summation orders, against
    60-digit arithmetic: its worst error is between 3e-8 and 1e-6 of the scale on every family of rows (the parity
    tests allow 2e-6), also where dy and the dot product cancel. A scale ten times too large or too small, or one
    without its dot-product term, leaves that band."""
    import mpmath as mp
    from oracle import fno
    rng = np.random.default_rng(11)
    with mp.workdps(60):
        for rows, cols, sigma, shift, scale in ((4, 257, 1.0, 0.0, 1.0), (3, 64, 3.0, 0.0, 0.125), (3, 1000, 1.0, 0.0, -0.5),
                                                (3, 96, 0.05, 7.0, 1.0), (3, 96, 0.01, -50.0, 2.0)):
            y = fso.softmax_f64(rng.standard_normal((rows, cols)).astype(np.float32) * 2, FP32, 1.0).astype(np.float32)
            dy = (rng.standard_normal((rows, cols)) * sigma + shift).astype(np.float32)      # shift: dy - dot nearly cancels
            want = np.empty((rows, cols))
            for i in range(rows):
                g = [mp.mpf(float(v)) for v in dy[i]]
                p = [mp.mpf(float(v)) for v in y[i]]
                dot = mp.fsum([a * b for a, b in zip(g, p)])
                want[i] = [float(mp.mpf(float(np.float32(scale))) * b * (a - dot)) for a, b in zip(g, p)]
            es = fno.backward_error_scale(dy, y, FP32, scale)
            worst = 0.0
            for order in (range(cols), range(cols - 1, -1, -1), np.random.default_rng(cols).permutation(cols)):
                got = np.empty_like(dy)
                for i in range(rows):
                    dot = np.float32(0)
                    for j in order:
                        dot = np.float32(dot + np.float32(dy[i, j] * y[i, j]))
                    got[i] = ((dy[i] - dot).astype(np.float32) * y[i]).astype(np.float32) * np.float32(scale)
                with np.errstate(invalid="ignore", divide="ignore"):
                    ratio = np.where(es > 0, np.abs(got - want) / es, 0.0)
                worst = max(worst, float(ratio.max()))
            assert 3e-8 <= worst <= 1e-6, (rows, cols, sigma, shift, scale, worst)
