"""Pins for the fp64 oracle: every check takes its expected value from something other than the
oracle itself -- a closed form, 100-digit mpmath arithmetic, exact rational arithmetic, a library
routine, or an invariant of the definition y_j = exp(z_j - max z) / sum_k exp(z_k - max z),
z = scale * x (the operator named in the paper's abstract and Sec. IV-C; the paper prints no
worked softmax example, so no printed values exist to quote).

CPU only.
"""
import itertools
import math
import os
from fractions import Fraction

import mpmath
import numpy as np
import pytest

from oracle import fso
from paper_2607_24762_b200 import workloads as W

FP32, BF16, FP16 = fso.FP32, fso.BF16, fso.FP16
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def ulps64(a, b):
    """Distance in fp64 units in the last place between finite non-negative arrays."""
    ia = np.asarray(a, dtype=np.float64).view(np.int64)
    ib = np.asarray(b, dtype=np.float64).view(np.int64)
    return np.abs(ia - ib)


def mp_softmax(row, scale=1.0):
    """The definition, at 100 significant digits; -inf entries contribute exactly 0."""
    with mpmath.workdps(100):
        z = [mpmath.mpf(float(scale)) * mpmath.mpf(float(v)) if np.isfinite(v) else None for v in row]
        finite = [v for v in z if v is not None]
        m = max(finite)
        e = [mpmath.exp(v - m) if v is not None else mpmath.mpf(0) for v in z]
        s = mpmath.fsum(e)
        return [float(v / s) for v in e]


# ---------------------------------------------------------------------------------------------
# brute force on tiny rows
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("cols", [1, 2, 3, 4])
def test_bruteforce_tiny_rows_vs_mpmath(cols):
    values = [-np.inf, -2.0, -0.5, 0.0, 1.0, 3.0]
    rows = [r for r in itertools.product(values, repeat=cols) if any(np.isfinite(v) for v in r)]
    x = np.array(rows, dtype=np.float32)
    y = fso.softmax_f64(x, FP32, 1.0)
    for r, row in enumerate(rows):
        want = np.array(mp_softmax(row))
        assert ulps64(y[r], want).max() <= 2, (row, y[r], want)
        for j, v in enumerate(row):
            if v == -np.inf:
                assert y[r, j] == 0.0 and not np.signbit(y[r, j])


def test_bruteforce_five_columns_sampled_vs_mpmath():
    values = [-np.inf, -7.25, -1.0, 0.0, 0.5, 2.0, 11.0]
    rows = list(itertools.product(values, repeat=5))[::37]
    rows = [r for r in rows if any(np.isfinite(v) for v in r)]
    x = np.array(rows, dtype=np.float32)
    for scale in (1.0, 0.25, -1.5):
        rows_s = rows
        if scale < 0:   # a negative scale turns -inf into +inf (NaN row); keep finite rows only
            rows_s = [r for r in rows if all(np.isfinite(v) for v in r)]
        xs = np.array(rows_s, dtype=np.float32)
        y = fso.softmax_f64(xs, FP32, scale)
        for r, row in enumerate(rows_s):
            want = np.array(mp_softmax(row, scale))
            assert ulps64(y[r], want).max() <= 2, (scale, row)
    assert x.shape[1] == 5


def test_golden_rows_from_mpmath_fixture():
    """tests/golden/softmax_mpmath.txt: inputs and 100-digit results written by make_mpmath_golden.py."""
    path = os.path.join(GOLDEN, "softmax_mpmath.txt")
    n = 0
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            dtype_s, scale_s, xs, ys = line.split("|")
            dtype = {"fp32": FP32, "bf16": BF16, "fp16": FP16}[dtype_s.strip()]
            scale = float.fromhex(scale_s.strip())
            xv = np.array([float.fromhex(t) for t in xs.split()], dtype=np.float64)
            want = np.array([float.fromhex(t) for t in ys.split()], dtype=np.float64)
            stored = W.to_stored(xv, dtype)
            # the fixture's inputs are exactly representable in their dtype
            assert np.array_equal(W.stored_to_f32(stored, dtype).astype(np.float64), xv)
            got = fso.softmax_f64(stored.reshape(1, -1), dtype, scale)[0]
            assert ulps64(got, want).max() <= 2, line[:60]
            n += 1
    assert n >= 12


# ---------------------------------------------------------------------------------------------
# closed forms and special cases
# ---------------------------------------------------------------------------------------------

def test_single_column_is_one():
    x = np.array([[0.0], [-3.5], [1e30], [-1e-30]], dtype=np.float32)
    assert np.array_equal(fso.softmax_f64(x, FP32, 1.0), np.ones((4, 1)))
    assert np.array_equal(fso.softmax_f64(x, FP32, -2.0), np.ones((4, 1)))


def test_two_columns_reduce_to_logistic():
    t = np.linspace(-30, 30, 241)
    x = np.stack([t, np.zeros_like(t)], axis=1).astype(np.float32)
    y = fso.softmax_f64(x, FP32, 1.0)
    tt = x[:, 0].astype(np.float64)
    sig = 1.0 / (1.0 + np.exp(-tt))
    sig2 = 0.5 * (1.0 + np.tanh(tt / 2.0))
    assert np.allclose(y[:, 0], sig, rtol=4e-16, atol=0)
    assert np.allclose(y[:, 0], sig2, rtol=0, atol=3e-16)
    assert np.allclose(y[:, 1], 1.0 / (1.0 + np.exp(tt)), rtol=4e-16, atol=0)


@pytest.mark.parametrize("cols", [1, 2, 3, 7, 128, 1000, 4096, 65537])
@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_uniform_row_is_exactly_one_over_n(cols, dtype):
    for value in (0.0, -1.75, 12.0):
        x = W.to_stored(np.full((2, cols), value), dtype)
        y = fso.softmax_f64(x, dtype, 0.5)
        assert np.all(y == 1.0 / cols)


def test_scale_zero_gives_uniform():
    x = W.random_case(3, 17, FP32, seed=5, sigma=10.0)
    assert np.all(fso.softmax_f64(x, FP32, 0.0) == 1.0 / 17)
    xi = x.copy()
    xi[1, 4] = -np.inf            # 0 * inf = NaN poisons that row only
    y = fso.softmax_f64(xi, FP32, 0.0)
    assert np.all(np.isnan(y[1])) and np.all(y[0] == 1.0 / 17) and np.all(y[2] == 1.0 / 17)


def test_rows_sum_to_one():
    for dtype, cols, sigma in [(FP32, 1000, 1.0), (BF16, 2048, 3.0), (FP16, 4097, 2.0), (FP32, 1 << 18, 4.0)]:
        x = W.random_case(3, cols, dtype, seed=11, sigma=sigma)
        y = fso.softmax_f64(x, dtype, 1.0)
        for r in range(3):
            assert abs(math.fsum(y[r]) - 1.0) <= 1e-14


def test_shift_invariance_is_bit_exact_on_a_dyadic_grid():
    rng = np.random.default_rng(3)
    base = rng.integers(-256, 256, size=(4, 333)) / 16.0          # multiples of 1/16, |x| <= 16
    x0 = base.astype(np.float32)
    y0 = fso.softmax_f64(x0, FP32, 1.0)
    for c in (-1024.0, 0.0625, 77.5, 4096.0):
        xc = (base + c).astype(np.float32)
        assert np.array_equal(xc.astype(np.float64), base + c)     # shift is exact in fp32
        assert np.array_equal(fso.softmax_f64(xc, FP32, 1.0), y0)


def test_power_of_two_scale_equals_prescaled_input():
    rng = np.random.default_rng(4)
    base = rng.integers(-512, 512, size=(3, 257)) / 8.0
    for k in (-3, -1, 1, 4):
        s = 2.0 ** k
        a = fso.softmax_f64(base.astype(np.float32), FP32, s)
        b = fso.softmax_f64((base * s).astype(np.float32), FP32, 1.0)
        assert np.array_equal(a, b)
    # sign: softmax(-1 * x) == softmax of the negated input
    a = fso.softmax_f64(base.astype(np.float32), FP32, -1.0)
    b = fso.softmax_f64((-base).astype(np.float32), FP32, 1.0)
    assert np.array_equal(a, b)


def test_scale_is_the_float_that_was_passed():
    """scale is a C float: 0.1f, not 0.1. The expected value uses the widened float."""
    x = np.array([[1.0, 2.0, 4.0, 8.0]], dtype=np.float32)
    s32 = float(np.float32(0.1))
    want = np.array(mp_softmax(x[0], s32))
    wrong = np.array(mp_softmax(x[0], 0.1))
    got = fso.softmax_f64(x, FP32, 0.1)[0]
    assert ulps64(got, want).max() <= 2
    assert ulps64(got, wrong).max() > 1000


def test_dominant_entry_saturates_to_one_hot():
    for dtype in (FP32, BF16, FP16):
        v = np.zeros((1, 50))
        v[0, 17] = 1000.0
        y = fso.softmax_f64(W.to_stored(v, dtype), dtype, 1.0)
        want = np.zeros((1, 50))
        want[0, 17] = 1.0
        assert np.array_equal(y, want)


def test_neg_inf_entries_are_exact_zero_and_do_not_disturb_the_rest():
    x = W.random_case(6, 301, FP32, seed=21, sigma=2.0, neg_inf_frac=0.4)
    y = fso.softmax_f64(x, FP32, 1.0)
    for r in range(x.shape[0]):
        masked = np.isneginf(x[r])
        assert masked.any() and (~masked).any()
        assert np.all(y[r, masked] == 0.0) and not np.any(np.signbit(y[r, masked]))
        sub = fso.softmax_f64(x[r, ~masked].reshape(1, -1), FP32, 1.0)[0]
        assert np.array_equal(y[r, ~masked], sub)        # sub-row consistency, bit-exact


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_nan_rules(dtype):
    def store(v):
        return W.to_stored(np.array(v, dtype=np.float64), dtype)
    ninf, pinf, nan = -np.inf, np.inf, np.nan
    y = fso.softmax_f64(store([[ninf, ninf, ninf]]), dtype, 1.0)
    assert np.all(np.isnan(y))                            # fully masked row
    y = fso.softmax_f64(store([[0.0, pinf, 1.0]]), dtype, 1.0)
    assert np.all(np.isnan(y))                            # +inf anywhere
    for pos in range(3):
        row = [0.5, -1.0, 2.0]
        row[pos] = nan
        assert np.all(np.isnan(fso.softmax_f64(store([row]), dtype, 1.0)))
    y = fso.softmax_f64(store([[0.0, ninf, 1.0]]), dtype, -1.0)
    assert np.all(np.isnan(y))                            # -1 * -inf = +inf
    # NaN rows do not leak into their neighbours
    y = fso.softmax_f64(store([[0.0, 1.0], [nan, 1.0], [0.0, 1.0]]), dtype, 1.0)
    assert np.all(np.isnan(y[1])) and np.array_equal(y[0], y[2]) and not np.isnan(y[0]).any()


def test_monotone_and_permutation_equivariant():
    x = W.random_case(4, 513, FP32, seed=8, sigma=3.0)
    y = fso.softmax_f64(x, FP32, 0.7)
    for r in range(4):
        order = np.argsort(x[r], kind="stable")
        assert np.all(np.diff(y[r, order]) >= 0)
    perm = np.random.default_rng(9).permutation(513)
    yp = fso.softmax_f64(np.ascontiguousarray(x[:, perm]), FP32, 0.7)
    assert ulps64(yp, y[:, perm]).max() <= 2


def test_negative_scale_reverses_order():
    x = W.random_case(2, 100, FP32, seed=10, sigma=2.0)
    y = fso.softmax_f64(x, FP32, -0.5)
    for r in range(2):
        order = np.argsort(x[r], kind="stable")
        assert np.all(np.diff(y[r, order]) <= 0)


def test_log_softmax_identity_against_scipy_logsumexp():
    from scipy.special import logsumexp, softmax as sp_softmax
    x = W.random_case(5, 777, FP32, seed=12, sigma=2.0)
    scale = float(np.float32(0.37))
    z = x.astype(np.float64) * scale
    y = fso.softmax_f64(x, FP32, 0.37)
    lse = logsumexp(z, axis=1, keepdims=True)
    assert np.abs(np.log(y) - (z - lse)).max() <= 1e-13
    assert np.abs(y - sp_softmax(z, axis=1)).max() <= 1e-15


def test_agrees_with_torch_fp64_eager_semantics():
    """Secondary witness: the paper's validator compares with eager framework output (Sec. III-C)."""
    import torch
    w = W.WORKLOADS["cfg1"]
    x = W.generate(w)
    y = fso.softmax_f64(x, FP32, w.scale)
    yt = torch.softmax(torch.from_numpy(x).double() * w.scale_f32, dim=-1).numpy()
    assert np.abs(y - yt).max() <= 1e-15
    special = np.array([[0.0, -np.inf, 1.0, 2.0], [-np.inf] * 4, [0.0, np.inf, 1.0, 2.0],
                        [np.nan, 0.0, 0.0, 0.0]], dtype=np.float32)
    ys = fso.softmax_f64(special, FP32, 1.0)
    yts = torch.softmax(torch.from_numpy(special).double(), dim=-1).numpy()
    assert np.array_equal(np.isnan(ys), np.isnan(yts))
    assert np.array_equal(ys == 0.0, yts == 0.0)


def test_compensated_sum_survives_many_small_terms():
    """One entry at 0 and 2^20 entries at -40: S = 1 + 2^20 * e^-40 exactly representable to 1e-30;
    a naive left-to-right fp64 sum starting from the 1 would drop every small term."""
    n = 1 << 20
    v = np.full((1, n + 1), -40.0)
    v[0, 0] = 0.0
    y = fso.softmax_f64(v.astype(np.float32), FP32, 1.0)
    with mpmath.workdps(60):
        em40 = mpmath.exp(-40)
        s = 1 + n * em40
        assert abs(y[0, 0] - float(1 / s)) <= 2.3e-16
        assert abs(y[0, 1] - float(em40 / s)) <= float(em40 / s) * 4e-16


# ---------------------------------------------------------------------------------------------
# stored-format decoders, rounding and the comparator
# ---------------------------------------------------------------------------------------------

def test_widen_matches_independent_decoders_for_every_16bit_pattern():
    import ml_dtypes
    bits = np.arange(65536, dtype=np.uint16)
    a = fso.widen(bits, FP16)
    b = bits.view(np.float16).astype(np.float64)
    assert np.array_equal(np.isnan(a), np.isnan(b)) and np.array_equal(a[~np.isnan(a)], b[~np.isnan(b)])
    a = fso.widen(bits, BF16)
    b = bits.view(ml_dtypes.bfloat16).astype(np.float64)
    assert np.array_equal(np.isnan(a), np.isnan(b)) and np.array_equal(a[~np.isnan(a)], b[~np.isnan(b)])
    f = np.array([1.5, -0.0, 3e38, 1e-45], dtype=np.float32)
    assert np.array_equal(fso.widen(f, FP32), f.astype(np.float64))


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_rounding_round_trips_every_pattern_and_breaks_ties_to_even(dtype):
    bits = np.arange(0x8000, dtype=np.uint16)                 # non-negative patterns
    vals = fso.widen(bits, dtype)
    finite = np.isfinite(vals)
    assert np.array_equal(fso.round_from_f64(vals[finite], dtype), bits[finite])
    assert np.array_equal(fso.round_from_f64(-vals[finite], dtype), bits[finite] | 0x8000)
    fb, fv = bits[finite], vals[finite]
    lo, hi = fv[:-1], fv[1:]
    mid = (lo + hi) / 2.0                                     # exact in fp64
    r = fso.round_from_f64(mid, dtype)
    even = np.where(fb[:-1] % 2 == 0, fb[:-1], fb[1:])
    assert np.array_equal(r, even)
    assert np.array_equal(fso.round_from_f64(np.nextafter(mid, np.inf), dtype), fb[1:])
    assert np.array_equal(fso.round_from_f64(np.nextafter(mid, -np.inf), dtype), fb[:-1])


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_rounding_matches_exact_rational_nearest(dtype):
    """Nearest representable value by exact Fraction arithmetic over the neighbouring patterns."""
    rng = np.random.default_rng(17)
    bits = np.arange(0x8000, dtype=np.uint16)
    vals = fso.widen(bits, dtype)
    finite_bits = bits[np.isfinite(vals)]
    grid = vals[np.isfinite(vals)]
    top = 1.0
    samples = np.concatenate([rng.random(300) * top, 10.0 ** rng.uniform(-45, 0, 300)])
    got = fso.round_from_f64(samples, dtype)
    for v, g in zip(samples, got):
        k = int(np.searchsorted(grid, v))
        cands = [c for c in (k - 1, k) if 0 <= c < len(grid)]
        fv = Fraction(float(v))
        best = min(cands, key=lambda c: (abs(Fraction(float(grid[c])) - fv), int(finite_bits[c]) & 1))
        assert int(g) == int(finite_bits[best]), (v, g, finite_bits[best])


def test_generator_rounding_agrees_with_oracle_rounding():
    """Two independent fp64 -> bf16 nearest-even roundings (numpy bit trick vs the C++ comparator)."""
    rng = np.random.default_rng(23)
    v = np.concatenate([rng.standard_normal(200000) * 3.0, 10.0 ** rng.uniform(-42, 2, 50000)])
    bits = np.arange(0x7F7F, dtype=np.uint16)
    grid = fso.widen(bits, BF16)
    mids = (grid[:-1] + grid[1:]) / 2
    v = np.concatenate([v, mids, np.nextafter(mids, 0), np.nextafter(mids, np.inf)])
    assert np.array_equal(W.f64_to_bf16_bits(v), fso.round_from_f64(v, BF16))
    assert np.array_equal(W.to_stored(v, FP16), fso.round_from_f64(v, FP16))


def test_comparator_applies_the_stated_tolerances():
    want = np.array([0.25, 0.5, 0.0, 0.125, 1e-300, 0.0078125])
    exact16 = fso.round_from_f64(want, BF16)
    rep = fso.compare(exact16, BF16, want)
    assert rep.max_ulp == 0 and rep.ok(BF16) and rep.n_compared == 6
    off1 = exact16.copy(); off1[1] += 1
    assert fso.compare(off1, BF16, want).max_ulp == 1 and fso.compare(off1, BF16, want).ok(BF16)
    off2 = exact16.copy(); off2[3] -= 2
    rep = fso.compare(off2, BF16, want)
    assert rep.max_ulp == 2 and rep.worst_index == 3 and not rep.ok(BF16)
    nz = exact16.copy(); nz[2] = 1                              # oracle says exact +0, result is not
    assert fso.compare(nz, BF16, want).zero_mismatch == 1 and not fso.compare(nz, BF16, want).ok(BF16)
    mz = exact16.copy(); mz[2] = 0x8000                          # -0 is not the +0 bit pattern
    assert fso.compare(mz, BF16, want).zero_mismatch == 1
    nanned = exact16.copy(); nanned[0] = 0x7FC0
    assert fso.compare(nanned, BF16, want).nan_mismatch == 1
    wn = want.copy(); wn[0] = np.nan
    assert fso.compare(nanned, BF16, wn).nan_mismatch == 0 and fso.compare(nanned, BF16, wn).ok(BF16)
    neg = exact16.copy(); neg[0] |= 0x8000
    assert fso.compare(neg, BF16, want).negative == 1

    g32 = want.astype(np.float32)
    rep = fso.compare(g32, FP32, want)
    assert rep.ok(FP32) and rep.max_abs_err <= 1e-300
    g32b = g32.copy(); g32b[1] += np.float32(2e-6)
    rep = fso.compare(g32b, FP32, want)
    assert not rep.ok(FP32) and rep.worst_index == 1 and abs(rep.max_abs_err - 2e-6) < 1e-7
    g32c = g32.copy(); g32c[1] += np.float32(5e-7)
    assert fso.compare(g32c, FP32, want).ok(FP32)
    g32n = g32.copy(); g32n[4] = np.nan
    assert fso.compare(g32n, FP32, want).nan_mismatch == 1
    # fp16 subnormal spacing: 2^-24 steps below 2^-14
    w16 = np.array([3 * 2.0 ** -24, 2.0 ** -15])
    e16 = fso.round_from_f64(w16, FP16)
    assert list(e16) == [3, 0x0200]
    assert fso.compare(np.array([5, 0x0200], dtype=np.uint16), FP16, w16).max_ulp == 2


def test_comparator_fp32_exact_zero_and_sign_rules():
    """fp32 results: an oracle value of exactly +0 (a -inf input) must be met by the +0 bit pattern, and a
    softmax output never carries a sign; each of these fails the bar even where |delta| is far below 1e-6."""
    want = np.array([0.25, 0.0, 0.5, 0.0, 0.25])
    exact = want.astype(np.float32)
    rep = fso.compare(exact, FP32, want)
    assert rep.ok(FP32) and rep.zero_mismatch == 0 and rep.negative == 0 and rep.n_compared == 5
    tiny = exact.copy(); tiny[1] = np.float32(1e-45)             # the smallest subnormal is not +0
    rep = fso.compare(tiny, FP32, want)
    assert rep.zero_mismatch == 1 and rep.negative == 0 and rep.max_abs_err < 1e-44 and not rep.ok(FP32)
    mz = exact.copy(); mz[3] = np.float32(-0.0)                  # -0: wrong bit pattern, but no magnitude
    rep = fso.compare(mz, FP32, want)
    assert rep.zero_mismatch == 1 and rep.negative == 0 and rep.max_abs_err == 0.0 and not rep.ok(FP32)
    neg0 = exact.copy(); neg0[1] = np.float32(-1e-30)            # negative where the oracle has +0: both rules
    rep = fso.compare(neg0, FP32, want)
    assert rep.zero_mismatch == 1 and rep.negative == 1 and not rep.ok(FP32)
    neg = exact.copy(); neg[0] = np.float32(-1e-30)              # negative where the oracle is positive
    wneg = want.copy(); wneg[0] = 1e-30
    rep = fso.compare(neg, FP32, wneg)
    assert rep.negative == 1 and rep.zero_mismatch == 0 and rep.max_abs_err < 1e-6 and not rep.ok(FP32)
    both = exact.copy(); both[1] = np.float32(1e-45); both[3] = np.float32(-0.0); both[4] = np.float32(-0.25)
    rep = fso.compare(both, FP32, want)
    assert rep.zero_mismatch == 2 and rep.negative == 1
    # the same rules leave a correct result alone when the oracle value is tiny but not zero
    wt = np.array([1e-300, 0.5])
    assert fso.compare(np.array([0.0, 0.5], dtype=np.float32), FP32, wt).ok(FP32)


# ---------------------------------------------------------------------------------------------
# workload structure seen through the oracle
# ---------------------------------------------------------------------------------------------

def test_vocabulary_rows_put_one_eighth_on_each_spike():
    w = W.WORKLOADS["cfg4"]
    x = W.generate_rows(w, 0, 2)
    xf = W.stored_to_f32(x, BF16)
    y = fso.softmax_f64(x, BF16, w.scale)
    for r in range(2):
        spikes = np.flatnonzero(xf[r] == W.SPIKE_VALUE)
        assert len(spikes) == W.N_SPIKES
        ys = y[r, spikes]
        assert np.all(ys == ys[0]) and 0.1249 < ys[0] < 0.125
        rest = np.delete(y[r], spikes)
        assert rest.max() < 1e-5
        assert np.all(fso.round_from_f64(ys, BF16) == fso.round_from_f64(np.array([0.125]), BF16)[0])


def test_causal_rows_are_zero_above_the_diagonal():
    w = W.WORKLOADS["cfg5"]
    x = W.generate_rows(w, 0, 3)
    y = fso.softmax_f64(x, FP32, w.scale)
    assert y[0, 0] == 1.0 and np.all(y[0, 1:] == 0.0)
    for i in range(3):
        assert np.count_nonzero(y[i] == 0.0) == w.cols - 1 - i
        assert abs(math.fsum(y[i]) - 1.0) < 1e-15
    x = W.generate_rows(w, 20000, 20001)
    y = fso.softmax_f64(x, FP32, w.scale)
    assert np.all(y[0, 20001:] == 0.0) and np.all(y[0, :20001] > 0.0)
