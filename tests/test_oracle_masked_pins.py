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
