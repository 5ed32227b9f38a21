"""GPU parity of fs_softmax_masked against the fp64 oracle, element by element on seeded inputs,
through the C ABI. The bar: fp32 |error| <= 1e-6 + 2.5e-7 * Z * y, Z the largest finite |scale * x +
mask| of the row (the exponent is formed in binary32 before the maximum is taken off); bf16/fp16
within one unit in the last place of the correctly rounded fp64 value; exact +0 for masked columns."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fno, fso
from paper_2607_24762_b200 import workloads as W
from tests.gpu_util import np_to_torch_bits, torch_bits_to_np

pytestmark = pytest.mark.gpu
FP32, BF16, FP16 = W.FP32, W.BF16, W.FP16


@pytest.fixture(scope="module", autouse=True)
def built_library():
    from paper_2607_24762_b200 import _build
    _build.build_library()
    yield
    assert fs.fs_device_status() == fs.FS_OK


def make(batch, heads, q, k, dtype, seed, kind="causal"):
    rng = np.random.default_rng(seed)
    x = fso.round_from_f64(rng.standard_normal((batch * heads * q, k)) * 3.0, dtype)
    if kind == "causal":                                       # the last q rows of a k-column causal mask
        m = np.where(np.arange(k)[None, :] > (np.arange(q)[:, None] + k - q), -np.inf, 0.0)
        m = np.tile(m, (batch, 1))
    elif kind == "padding":                                    # per batch element, a padded tail
        m = np.zeros((batch * q, k))
        for b in range(batch):
            m[b * q:(b + 1) * q, k - 1 - (b * 7) % max(1, k // 2):] = -np.inf
        m[:, 0] = 0.0
    else:                                                      # a finite bias (ALiBi-like) plus some masked entries
        m = -np.abs(np.arange(k)[None, :] - np.arange(batch * q)[:, None] % k) * 0.0625
        m = np.where(rng.random((batch * q, k)) < 0.05, -np.inf, m)
        m[:, 0] = 0.0
    return x, fso.round_from_f64(m, dtype)


def run(x, mask, dtype, q, heads, scale, inplace=False, misalign=0):
    rows, cols = x.shape
    pad = lambda a: np.concatenate([np.zeros(misalign, a.dtype), a.ravel()])
    xd, md = np_to_torch_bits(pad(x)).cuda(), np_to_torch_bits(pad(mask)).cuda()
    yd = xd if inplace else torch.zeros_like(xd)
    off = misalign * W.ELEM_SIZE[dtype]
    fs.fs_softmax_masked(xd.data_ptr() + off, md.data_ptr() + off, yd.data_ptr() + off, rows, cols, q, heads, dtype, scale,
                         torch.cuda.current_stream())
    torch.cuda.synchronize()
    return torch_bits_to_np(yd, dtype)[misalign:].reshape(rows, cols)


def check(x, mask, dtype, q, heads, scale, **kw):
    got = run(x, mask, dtype, q, heads, scale, **kw)
    want = fso.softmax_masked_f64(x, mask, dtype, q, heads, scale)
    bound = fno.masked_softmax_bound(x, mask, dtype, q, heads, scale, want)      # pinned in tests/test_oracle_masked_pins.py
    rep = fno.compare(got, dtype, want, bound, rel_tol=1.0)
    assert rep.ok(dtype, rel_tol=1.0), (x.shape, dtype, scale, rep)
    g64 = fso.widen(got, dtype)
    assert np.all(g64[want == 0.0] == 0.0)                     # masked columns are exactly +0
    assert not np.any(np.signbit(g64[g64 == 0.0]))
    return rep


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_attention_shapes(dtype):
    for ci, (batch, heads, q, k, kind) in enumerate([(1, 1, 1, 8, "causal"), (2, 3, 4, 16, "causal"), (1, 2, 64, 64, "causal"),
                                                     (2, 4, 33, 128, "padding"), (1, 8, 128, 1024, "causal"), (2, 2, 16, 2048, "bias"),
                                                     (1, 2, 8, 4096, "padding"), (1, 2, 6, 5000, "bias"), (1, 1, 5, 32768, "causal"),
                                                     (1, 2, 3, 100000, "padding"), (1, 1, 2, 262144, "bias"), (2, 1, 3, 1001, "causal")]):
        x, m = make(batch, heads, q, k, dtype, seed=600 + ci, kind=kind)
        check(x, m, dtype, q, heads, [1.0, 0.125, 128 ** -0.5, -0.5][ci % 4])


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_row_lengths_across_the_split_geometries(dtype):
    esz = W.ELEM_SIZE[dtype]
    for kb, q in ((6, 300), (8, 800), (12, 500), (24, 300), (40, 200), (96, 100), (100, 80), (160, 60), (250.5, 40), (384, 30), (600, 16),
                  (1024, 8), (2048, 3)):
        k = int(kb * 1024) // esz
        x, m = make(1, 2, q, k, dtype, seed=int(kb), kind="padding")
        check(x, m, dtype, q, 2, 0.25)


@pytest.mark.parametrize("dtype", [BF16, FP16, FP32])
def test_rows_around_the_four_rows_per_block_kernel(dtype):
    """16-bit rows of 256..640 sixteen-byte vectors take the kernel that works on four rows per block from
    shared memory: both ends of that range and one vector beyond them, row counts that leave a block
    partly empty, every mask kind."""
    ve = 16 // W.ELEM_SIZE[dtype]
    for ci, nvec in enumerate((255, 256, 257, 400, 639, 640, 641)):
        for heads, q in ((1, 1), (1, 5), (3, 7), (2, 65)):
            x, m = make(1, heads, q, nvec * ve, dtype, seed=900 + ci * 7 + q, kind=("causal", "padding", "bias")[(ci + q) % 3])
            check(x, m, dtype, q, heads, [1.0, 0.25, -0.5][(ci + heads) % 3])


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_masks_shared_by_many_heads(dtype):
    """16-bit rows of 256..704 vectors with masks shared by 2 to 16 heads over one to three batches: head counts
    around the four rows a block takes, both ends of the row range, every mask kind, in place, special values."""
    ve = 8
    for ci, (batch, heads, q, nvec) in enumerate([(1, 2, 9, 256), (2, 4, 5, 256), (1, 3, 17, 300), (2, 5, 3, 512), (1, 8, 6, 640),
                                                   (3, 7, 2, 704), (1, 16, 1, 257), (1, 2, 130, 384), (1, 4, 33, 703)]):
        x, m = make(batch, heads, q, nvec * ve, dtype, seed=1200 + ci, kind=("causal", "padding", "bias")[ci % 3])
        check(x, m, dtype, q, heads, [1.0, 0.125, -0.5, 128 ** -0.5][ci % 4], inplace=ci % 4 == 3)
    # a fully masked row, a NaN and a +inf: whole rows NaN, the other heads of the block untouched
    x, m = make(1, 4, 3, 2048, dtype, seed=1300, kind="padding")
    ninf = np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    m[1, :] = ninf
    x[0, 7] = np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    x[5, 100] = np.uint16(0x7F80 if dtype == BF16 else 0x7C00)
    got = run(x, m, dtype, 3, 4, 1.0)
    want = fso.softmax_masked_f64(x, m, dtype, 3, 4, 1.0)
    assert np.array_equal(np.isnan(fso.widen(got, dtype)), np.isnan(want))
    ok = ~np.isnan(want).any(axis=1)
    assert fso.compare(got[ok], dtype, want[ok]).ok(dtype)
    # bf16 results below 2^-126 are kept (the 1-ulp rule covers subnormals)
    if dtype == BF16:
        row = np.linspace(-91.0, -87.0, 2048)
        row[0] = 0.0
        xs = fso.round_from_f64(np.tile(row, (4, 1)), dtype)
        ms = fso.round_from_f64(np.zeros((2, 2048)), dtype)
        rep = check(xs, ms, dtype, 2, 2, 1.0)
        y = run(xs, ms, dtype, 2, 2, 1.0)
        assert np.count_nonzero((y[0] > 0) & (y[0] < 0x0080)) > 50


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_special_values_alignment_and_aliasing(dtype):
    x, m = make(1, 2, 4, 4096, dtype, seed=9, kind="padding")
    ninf = np.float32(-np.inf) if dtype == FP32 else np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    nan = np.float32(np.nan) if dtype == FP32 else np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    m[1, :] = ninf                                             # a fully masked row: NaN
    x[2, 5] = nan
    got = run(x, m, dtype, 4, 2, 1.0)
    want = fso.softmax_masked_f64(x, m, dtype, 4, 2, 1.0)
    assert np.array_equal(np.isnan(fso.widen(got, dtype)), np.isnan(want))
    x, m = make(1, 2, 16, 2048, dtype, seed=10, kind="causal")
    check(x, m, dtype, 16, 2, 0.5, inplace=True)
    x, m = make(1, 2, 5, 1024, dtype, seed=11, kind="bias")
    check(x, m, dtype, 5, 2, 0.5, misalign=1)
    fs.fs_softmax_masked(None, None, None, 0, 128, 1, 1, dtype)
    L = fs.binding.lib()
    a, b, c = 0x10000, 0x2000000, 0x4000000
    assert L.fs_softmax_masked(a, c, b, 8, 8, 3, 1, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG       # rows not a multiple
    assert L.fs_softmax_masked(a, None, b, 8, 8, 4, 2, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG
    assert L.fs_softmax_masked(a, c, b, 8, 8, 0, 2, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG


def test_attention_workload_full_size():
    """cfg2's shape as (1 batch, 8 heads, 2048 queries) x 2048 keys with a causal mask shared by the heads."""
    w = W.WORKLOADS["cfg2"]
    x = W.generate_rows(w, 0, w.rows)
    m = fso.round_from_f64(np.where(np.arange(2048)[None, :] > np.arange(2048)[:, None], -np.inf, 0.0), w.dtype)
    rep = check(x, m, w.dtype, 2048, 8, w.scale_f32)
    print("cfg2 masked", rep)
