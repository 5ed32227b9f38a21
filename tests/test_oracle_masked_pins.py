"""Pins for the oracle's additive-mask softmax: 100-digit mpmath on small cases, PyTorch float64 with
broadcasting over heads, reduction to the pinned plain and causal oracles, loops for the row mapping.
CPU only."""
import mpmath
import numpy as np
import torch

from oracle import fso

FP32, BF16 = fso.FP32, fso.BF16


def test_small_cases_vs_mpmath_and_row_mapping():
    rng = np.random.default_rng(6)
    batch, heads, q, k = 2, 3, 4, 5
    x = (rng.integers(-40, 40, size=(batch * heads * q, k)) / 8).astype(np.float32)
    mask = (rng.integers(-16, 1, size=(batch * q, k)) / 4).astype(np.float32)
    mask[1, 2] = -np.inf
    for scale in (1.0, 0.5, -0.25):
        y = fso.softmax_masked_f64(x, mask, FP32, q, heads, scale)
        sc = float(np.float32(scale))
        for b in range(batch):
            for h in range(heads):
                for i in range(q):
                    row = (b * heads + h) * q + i
                    with mpmath.workdps(100):
                        z = [mpmath.mpf(sc) * mpmath.mpf(float(x[row, j])) + (mpmath.mpf(float(mask[b * q + i, j])) if np.isfinite(mask[b * q + i, j]) else mpmath.mpf("-inf"))
                             for j in range(k)]
                        m = max(z)
                        e = [mpmath.exp(v - m) if v != mpmath.mpf("-inf") else mpmath.mpf(0) for v in z]
                        s = mpmath.fsum(e)
                        want = np.array([float(v / s) for v in e])
                    assert np.max(np.abs(y[row] - want)) < 1e-15


def test_against_torch_float64_broadcast():
    g = torch.Generator().manual_seed(2)
    batch, heads, q, k = 2, 4, 16, 33
    x = torch.randn(batch, heads, q, k, generator=g) * 3
    mask = torch.randn(batch, 1, q, k, generator=g)
    mask[mask < -1.0] = float("-inf")
    mask[:, :, :, 0] = 0.0                                   # never a fully masked row
    want = torch.softmax(x.double() * 0.125 + mask.double(), -1).reshape(-1, k).numpy()
    got = fso.softmax_masked_f64(x.reshape(-1, k).numpy(), mask.reshape(-1, k).numpy(), FP32, q, heads, 0.125)
    assert np.max(np.abs(got - want)) < 1e-15


def test_reduces_to_the_plain_and_causal_oracles():
    rng = np.random.default_rng(3)
    q = k = 24
    x = rng.standard_normal((2 * q, k)).astype(np.float32)
    zero = np.zeros((q, k), dtype=np.float32)
    assert np.array_equal(fso.softmax_masked_f64(x, zero, FP32, q, 2, 0.7), fso.softmax_f64(x, FP32, 0.7))
    causal = np.where(np.arange(k)[None, :] > np.arange(q)[:, None], -np.inf, 0.0).astype(np.float32)
    assert np.array_equal(fso.softmax_masked_f64(x, causal, FP32, q, 2, 0.7), fso.softmax_causal_f64(x.reshape(2, q, k)[0], FP32, 0, 0.7).tolist() + fso.softmax_causal_f64(x.reshape(2, q, k)[1], FP32, 0, 0.7).tolist())
    # a fully masked row is NaN; a constant mask row changes nothing
    m = zero.copy(); m[3, :] = -np.inf; m[5, :] = 2.5
    y = fso.softmax_masked_f64(x, m, FP32, q, 2, 1.0)
    assert np.all(np.isnan(y[3])) and np.all(np.isnan(y[q + 3]))
    assert np.max(np.abs(y[5] - fso.softmax_f64(x, FP32, 1.0)[5])) < 1e-15


# ---------------------------------------------------------------------------------------------
# masked_softmax_bound: the fp32 tolerance of the masked entry point's parity tests
# ---------------------------------------------------------------------------------------------

def test_masked_bound_hand_computed():
    from oracle import fno
    x = np.array([[1.0, -2.0], [4.0, 0.5], [0.0, 8.0], [-16.0, 2.0]], dtype=np.float32)          # 2 heads x 2 queries
    m = np.array([[0.0, -np.inf], [-1.0, 3.0]], dtype=np.float32)                                  # shared by the heads
    want = np.array([[1.0, 0.0], [0.25, 0.75], [1.0, 0.0], [0.5, 0.5]])
    b = fno.masked_softmax_bound(x, m, FP32, 2, 2, 0.5, want)
    # Z per row (finite |0.5 x + mask| only): row 0: |0.5|; row 1: max(|2 - 1|, |0.25 + 3|) = 3.25; row 2: 0 (4 - inf is
    # not finite); row 3: max(|-8 - 1|, |1 + 3|) = 9
    expect = 1e-6 + 2.5e-7 * np.array([[0.5], [3.25], [0.0], [9.0]]) * want
    assert np.allclose(b, expect, rtol=1e-15, atol=0)


def test_masked_bound_brackets_a_binary32_evaluation():
    """The arithmetic the entry point documents -- exponent scale * x + mask formed in binary32, maximum taken off, base-2
    exponential, binary32 sum, one division -- carried out in numpy float32 against 60-digit arithmetic: the worst error
    is between 2 % and 100 % of the bound, for exponents of a few units and for exponents in the hundreds (where the
    bound's second term is fifty times its first). A bound ten times looser, or without its Z term, fails."""
    import mpmath as mp
    from oracle import fno
    rng = np.random.default_rng(21)
    with mp.workdps(60):
        for heads, q, k, sigma, bias, scale in ((2, 3, 257, 2.0, 0.0, 1.0), (1, 4, 64, 3.0, 0.0, 0.125), (2, 2, 500, 1.0, 200.0, 1.0),
                                                (1, 3, 128, 0.5, -400.0, 1.0), (2, 2, 96, 2.0, 30.0, -1.0)):
            x = (rng.standard_normal((heads * q, k)) * sigma).astype(np.float32)
            m = (rng.standard_normal((q, k)) * 0.5 + bias).astype(np.float32)
            m[:, ::7] = -np.inf
            m[:, 0] = np.float32(bias)
            want = fso.softmax_masked_f64(x, m, FP32, q, heads, scale)
            bound = fno.masked_softmax_bound(x, m, FP32, q, heads, scale, want)
            mrow = np.arange(heads * q) % q
            c = np.float32(np.float64(np.float32(scale)) * 1.4426950408889634)
            l2e = np.float32(1.4426950408889634)
            t = (x * c).astype(np.float32) + (m[mrow] * l2e).astype(np.float32)                      # two roundings where the kernel fuses: not better
            t = t.astype(np.float32)
            r = t.max(axis=1, keepdims=True)
            e = np.exp2((t - r).astype(np.float32)).astype(np.float32)
            worst = 0.0
            for order in (np.arange(k), np.arange(k)[::-1], np.random.default_rng(k).permutation(k)):
                ssum = np.zeros(heads * q, dtype=np.float32)
                for j in order:
                    ssum = (ssum + e[:, j]).astype(np.float32)
                got = (e / ssum[:, None]).astype(np.float32)
                worst = max(worst, float(np.max(np.abs(got.astype(np.float64) - want) / bound)))
            assert 0.02 <= worst <= 1.0, (heads, q, k, sigma, bias, scale, worst)
