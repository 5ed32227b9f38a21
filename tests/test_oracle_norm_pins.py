"""Pins for the normalisation oracle (oracle/fno.py): expected values come from stored 60-digit mpmath
evaluations, PyTorch's float64 CPU operators (an independent library), closed forms, invariants and a
pure-Python loop over a tiny tensor -- never from the oracle itself. CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fno, fso
from paper_2607_24762_b200 import workloads as W

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "norm_mpmath.txt")


def read_golden():
    cases = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        kind, groups, shape, eps, x, gamma, beta, y = [f.strip() for f in line.split("|")]
        hx = lambda s: None if s == "-" else np.array([float.fromhex(t) for t in s.split()])
        cases.append((kind, int(groups), tuple(int(v) for v in shape.split(",")), float.fromhex(eps), hx(x), hx(gamma),
                      hx(beta), hx(y)))
    return cases


def f32(a):
    return None if a is None else np.asarray(a, dtype=np.float32)


def test_golden_mpmath_values():
    cases = read_golden()
    assert len(cases) >= 8
    for kind, groups, (n, ch, sp), eps, x, gamma, beta, want in cases:
        if kind == "layer":
            got = fno.layer_norm_f64(f32(x).reshape(n, sp), FP32, f32(gamma), f32(beta), eps).ravel()
        else:
            got = fno.group_norm_f64(f32(x).reshape(n, ch, sp), FP32, groups, f32(gamma), f32(beta), eps).ravel()
        scale = np.maximum(1.0, np.abs(want))
        assert np.max(np.abs(got - want) / scale) < 1e-13, (kind, groups, (n, ch, sp))


@pytest.mark.parametrize("dtype,tdt", [(FP32, torch.float32), (BF16, torch.bfloat16), (FP16, torch.float16)])
def test_layer_norm_against_torch_float64(dtype, tdt):
    g = torch.Generator().manual_seed(5 + dtype)
    for rows, cols, affine in ((1, 1, True), (3, 7, True), (5, 64, False), (2, 1000, True), (4, 4097, True)):
        xt = (torch.randn(rows, cols, generator=g) * 3 + 1.5).to(tdt)
        gt = (torch.randn(cols, generator=g)).to(tdt) if affine else None
        bt = (torch.randn(cols, generator=g)).to(tdt) if affine else None
        eps = 1e-5
        want = torch.nn.functional.layer_norm(xt.double(), (cols,), None if gt is None else gt.double(),
                                              None if bt is None else bt.double(), float(np.float32(eps))).numpy()
        to_np = lambda t: None if t is None else (t.numpy() if dtype == FP32 else t.view(torch.int16).numpy().view(np.uint16))
        got = fno.layer_norm_f64(to_np(xt), dtype, to_np(gt), to_np(bt), eps)
        assert np.max(np.abs(got - want)) < 1e-11 * max(1.0, float(np.max(np.abs(want))))


@pytest.mark.parametrize("dtype,tdt", [(FP32, torch.float32), (BF16, torch.bfloat16)])
def test_group_norm_against_torch_float64(dtype, tdt):
    g = torch.Generator().manual_seed(11 + dtype)
    for n, ch, sp, groups in ((1, 4, 6, 2), (2, 6, 5, 3), (3, 8, 16, 1), (2, 32, 9, 32), (1, 12, 64, 4)):
        xt = (torch.randn(n, ch, sp, generator=g) * 2 - 0.75).to(tdt)
        gt = torch.randn(ch, generator=g).to(tdt)
        bt = torch.randn(ch, generator=g).to(tdt)
        eps = 1e-5
        want = torch.nn.functional.group_norm(xt.double(), groups, gt.double(), bt.double(), float(np.float32(eps))).numpy()
        to_np = lambda t: t.numpy() if dtype == FP32 else t.view(torch.int16).numpy().view(np.uint16)
        got = fno.group_norm_f64(to_np(xt), dtype, groups, to_np(gt), to_np(bt), eps)
        assert np.max(np.abs(got - want)) < 1e-11 * max(1.0, float(np.max(np.abs(want))))


def test_group_norm_indexing_by_python_loops():
    """Channel c of sample s belongs to group c // (channels/groups); gamma/beta are indexed by c."""
    rng = np.random.default_rng(3)
    n, ch, sp, groups, eps = 2, 6, 5, 3, float(np.float32(1e-3))
    x = rng.integers(-20, 20, size=(n, ch, sp)).astype(np.float32) / 4
    gamma = rng.integers(-8, 8, size=ch).astype(np.float32) / 4
    beta = rng.integers(-8, 8, size=ch).astype(np.float32) / 2
    got = fno.group_norm_f64(x, FP32, groups, gamma, beta, eps)
    cpg = ch // groups
    for s in range(n):
        for gi in range(groups):
            vals = [float(x[s, c, k]) for c in range(gi * cpg, (gi + 1) * cpg) for k in range(sp)]
            mu = math.fsum(vals) / len(vals)
            var = math.fsum((v - mu) ** 2 for v in vals) / len(vals)
            for c in range(gi * cpg, (gi + 1) * cpg):
                for k in range(sp):
                    want = (float(x[s, c, k]) - mu) / math.sqrt(var + eps) * float(gamma[c]) + float(beta[c])
                    assert abs(got[s, c, k] - want) < 1e-13 * max(1.0, abs(want))


def test_closed_forms():
    # a constant row has zero variance: (x - mu) = 0, so y = beta exactly, whatever gamma and eps are
    x = np.full((2, 9), 3.25, dtype=np.float32)
    gamma = np.linspace(-2, 2, 9).astype(np.float32)
    beta = np.linspace(1, 5, 9).astype(np.float32)
    y = fno.layer_norm_f64(x, FP32, gamma, beta, 1e-5)
    assert np.array_equal(y, np.broadcast_to(beta.astype(np.float64), (2, 9)))
    # two elements a, b: mu = (a+b)/2, var = h^2 with h = (a-b)/2, y = +-h / sqrt(h^2 + eps)
    for a, b, eps in ((1.0, 3.0, 1e-5), (-2.5, 7.0, 0.25), (100.0, 100.5, 1e-6)):
        e = float(np.float32(eps))
        h = (a - b) / 2
        y = fno.layer_norm_f64(np.array([[a, b]], dtype=np.float32), FP32, None, None, eps)
        want = h / math.sqrt(h * h + e)
        assert abs(y[0, 0] - want) < 1e-15 and abs(y[0, 1] + want) < 1e-15
    # one element: x - mu = 0, y = beta
    y = fno.layer_norm_f64(np.array([[42.0]], dtype=np.float32), FP32, np.array([3.0], np.float32), np.array([-1.5], np.float32))
    assert y[0, 0] == -1.5
    # eps dominates: var = 1 (values -1, +1), eps = 3 gives y = +-1/2 exactly
    y = fno.layer_norm_f64(np.array([[-1.0, 1.0]], dtype=np.float32), FP32, None, None, 3.0)
    assert np.array_equal(y, [[-0.5, 0.5]])


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_invariants(dtype):
    x = W.random_case(6, 257, dtype, seed=21, sigma=2.0, neg_inf_frac=0.0)
    eps = 1e-5
    e = float(np.float32(eps))
    X = fso.widen(x, dtype)
    y = fno.layer_norm_f64(x, dtype, None, None, eps)
    var = X.var(axis=1)
    assert np.max(np.abs(y.sum(axis=1))) < 1e-10                                  # zero mean
    assert np.max(np.abs((y * y).sum(axis=1) - 257 * var / (var + e))) < 1e-9     # sum of squares
    # the order of the elements of a row is kept (monotone map)
    for i in range(6):
        assert np.array_equal(np.argsort(X[i], kind="stable"), np.argsort(y[i], kind="stable"))


def test_shift_and_scale_invariance():
    rng = np.random.default_rng(9)
    x = (rng.integers(-64, 64, size=(4, 33)) / 8).astype(np.float32)
    y0 = fno.layer_norm_f64(x, FP32, None, None, 1e-5)
    y1 = fno.layer_norm_f64((x + np.float32(16.0)).astype(np.float32), FP32, None, None, 1e-5)     # exact shifts
    assert np.max(np.abs(y0 - y1)) < 1e-13
    # with eps = 0 a positive factor cancels; a negative one flips the sign
    y2 = fno.layer_norm_f64(x, FP32, None, None, 0.0)
    y3 = fno.layer_norm_f64((x * np.float32(4.0)).astype(np.float32), FP32, None, None, 0.0)
    y4 = fno.layer_norm_f64((x * np.float32(-0.5)).astype(np.float32), FP32, None, None, 0.0)
    assert np.max(np.abs(y2 - y3)) < 1e-13 and np.max(np.abs(y2 + y4)) < 1e-13


def test_special_values_follow_ieee():
    x = np.array([[1.0, np.nan, 2.0], [1.0, np.inf, 2.0], [0.0, 0.0, 0.0]], dtype=np.float32)
    y = fno.layer_norm_f64(x, FP32, None, None, 1e-5)
    assert np.all(np.isnan(y[0])) and np.all(np.isnan(y[1]))
    assert np.array_equal(y[2], [0.0, 0.0, 0.0])
    assert fno.layer_norm_f64(np.zeros((0, 5), np.float32), FP32).shape == (0, 5)


def test_a_mutated_formula_fails_the_pins():
    """The pins see the usual mistakes: unbiased variance, eps outside the root, gamma/beta swapped."""
    x = np.array([[0.0, 1.0, 2.0, 3.0]], dtype=np.float32)
    kind, groups, shape, eps, gx, gg, gb, want = read_golden()[0]
    X = x.astype(np.float64)
    mu = X.mean()
    d = X - mu
    unbiased = d / np.sqrt((d * d).sum() / 3 + eps)
    eps_outside = d / (np.sqrt((d * d).mean()) + eps)
    for wrong in (unbiased, eps_outside):
        assert np.max(np.abs(wrong.ravel() - want)) > 1e-7


def test_comparator_rules():
    want = np.array([1.0, -2.0, 0.5, 1e-3])
    scale = np.array([1.0, 2.0, 0.5, 4.0])
    got = want.astype(np.float32)
    assert fno.compare(got, FP32, want, scale).ok(FP32)
    bad = got.copy(); bad[1] += np.float32(1e-4)
    assert not fno.compare(bad, FP32, want, scale).ok(FP32)
    nanned = got.copy(); nanned[0] = np.nan
    assert fno.compare(nanned, FP32, want, scale).nan_mismatch == 1
    # 16-bit: one unit off passes, two units off fails unless the fp32 bound covers it
    gb = fso.round_from_f64(want, BF16)
    assert fno.compare(gb, BF16, want, scale).ok(BF16)
    off1 = gb.copy(); off1[0] += 1
    assert fno.compare(off1, BF16, want, scale).ok(BF16)
    off2 = gb.copy(); off2[0] += 2
    assert not fno.compare(off2, BF16, want, scale).ok(BF16)
    off2s = gb.copy(); off2s[3] += 2         # |delta| = 2 ulp of 1e-3 ~ 1.5e-5 > 2e-6 * 4: still fails
    assert not fno.compare(off2s, BF16, want, scale).ok(BF16)
    big = np.array([4000.0, 4000.0, 4000.0, 4000.0])   # cancellation: a large scale excuses a small result's ulps
    assert fno.compare(off2s, BF16, want, big).ok(BF16)


# ---------------------------------------------------------------------------------------------
# error_scale: the magnitude the binary32 tolerance of the normalisation parity tests multiplies
# ---------------------------------------------------------------------------------------------

def test_error_scale_hand_computed_rows():
    """|gamma| (|x - mu| + mean|x|) / sqrt(var + eps) + |beta| worked out by hand."""
    x = np.array([[1.0, 3.0], [0.0, 4.0]], dtype=np.float32)
    # row 0: mu 2, var 1, mean|x| 2 -> (1 + 2) / 1 = 3; row 1: mu 2, var 4, mean|x| 2 -> (2 + 2) / 2 = 2
    s = fno.error_scale(x, FP32, x.shape, None, None, 0.0)
    assert np.array_equal(s, [[3.0, 3.0], [2.0, 2.0]])
    gamma = np.array([[2.0, -3.0]])
    beta = np.array([[0.5, -1.0]])
    s = fno.error_scale(x, FP32, x.shape, gamma, beta, 0.0)
    assert np.array_equal(s, [[6.5, 10.0], [4.5, 7.0]])
    assert np.array_equal(fno.error_scale(x, FP32, x.shape, gamma, None, 0.0), [[6.0, 9.0], [4.0, 6.0]])
    assert np.array_equal(fno.error_scale(x, FP32, x.shape, None, beta, 0.0), [[3.5, 4.0], [2.5, 3.0]])
    # eps sits under the root, next to the variance: var 1, eps 3 -> divisor 2
    assert np.array_equal(fno.error_scale(x[:1], FP32, (1, 2), None, None, 3.0), [[1.5, 1.5]])
    # a row far from zero: the mean term dominates (mu 1000, |d| 1, var 1)
    far = np.array([[999.0, 1001.0]], dtype=np.float32)
    assert np.array_equal(fno.error_scale(far, FP32, (1, 2), None, None, 0.0), [[1001.0, 1001.0]])
    # the view: six elements as 2 x 3 and as 3 x 2 are different rows
    six = np.array([0, 3, 6, 1, 1, 1], dtype=np.float32)
    s23 = fno.error_scale(six, FP32, (2, 3), None, None, 0.0)
    assert s23.shape == (2, 3) and np.allclose(s23[0], [(3 + 3) / math.sqrt(6), 3 / math.sqrt(6), (3 + 3) / math.sqrt(6)])


def _layer_norm_binary32(x, gamma, beta, eps, order):
    """layer_norm carried out in binary32, one rounding per operation, sums taken in `order`."""
    out = np.empty_like(x)
    one, n = np.float32(1), np.float32(x.shape[1])
    for i, row in enumerate(x):
        s = np.float32(0)
        for j in order:
            s = np.float32(s + row[j])
        mu = np.float32(s / n)
        d = (row - mu).astype(np.float32)
        q = np.float32(0)
        for j in order:
            q = np.float32(q + np.float32(d[j] * d[j]))
        rstd = np.float32(one / np.sqrt(np.float32(np.float32(q / n) + np.float32(eps))))
        out[i] = ((d * rstd).astype(np.float32) * gamma).astype(np.float32) + beta
    return out


def test_error_scale_brackets_a_binary32_evaluation():
    """The error of a plain binary32 layer_norm, measured against 60-digit arithmetic, is a fixed small multiple
    of error_scale whatever the row length, offset, spread or summation order: between 5e-8 and 1e-6 of it
    (binary32's unit roundoff is 6e-8; the parity tests allow 2e-6). A scale that is ten times too large or too
    small, or that drops the mean, gamma or beta term, leaves that band on at least one case."""
    import mpmath as mp
    rng = np.random.default_rng(7)
    with mp.workdps(60):
        for rows, cols, offset, spread, gscale, bscale in ((4, 257, 0.0, 1.0, 0.5, 1.0), (4, 64, 5.0, 0.5, 0.5, 1.0),
                                                           (3, 1000, -2.0, 3.0, 0.5, 1.0), (3, 96, 40.0, 1.0, 1.0, 0.0),
                                                           (3, 96, 0.0, 1.0, 20.0, 0.0), (3, 96, 0.0, 1.0, 0.01, 30.0)):
            x = (rng.standard_normal((rows, cols)) * spread + offset).astype(np.float32)
            gamma = (rng.standard_normal(cols) * gscale + gscale).astype(np.float32)
            beta = (rng.standard_normal(cols) * bscale).astype(np.float32)
            eps = 1e-5
            want = np.empty((rows, cols))
            for i in range(rows):
                xs = [mp.mpf(float(v)) for v in x[i]]
                mu = mp.fsum(xs) / cols
                sd = mp.sqrt(mp.fsum([(v - mu) ** 2 for v in xs]) / cols + mp.mpf(float(np.float32(eps))))
                want[i] = [float((v - mu) / sd * mp.mpf(float(gamma[j])) + mp.mpf(float(beta[j]))) for j, v in enumerate(xs)]
            scale = fno.error_scale(x, FP32, x.shape, gamma.astype(np.float64)[None, :], beta.astype(np.float64)[None, :], eps)
            worst = 0.0
            for order in (range(cols), range(cols - 1, -1, -1), np.random.default_rng(cols).permutation(cols)):
                got = _layer_norm_binary32(x, gamma, beta, eps, list(order))
                worst = max(worst, float(np.max(np.abs(got - want) / scale)))
            assert 5e-8 <= worst <= 1e-6, (rows, cols, offset, spread, gscale, bscale, worst)
