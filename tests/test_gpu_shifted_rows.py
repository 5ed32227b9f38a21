"""Rows whose byte length is not a multiple of 16, in tensors that are themselves 16-byte aligned: rows up to 512
bytes are taken 128 at a time as one contiguous span of the tensor (the span's first and last vector are shared with
the neighbouring blocks), longer ones by the block kernel, and beyond 16 KiB by the split-row kernel, on the aligned
vectors that cover each row (the first and last vector of a row are shared with its neighbours). Element-wise parity against the oracle with guard bands around the buffers: every head offset a row
can have, rows shorter than a vector, rows that end at the tensor's last partial vector, every dtype, negative
scales, in place, special values, and the row lengths on both sides of what a block's registers hold."""
import numpy as np
import pytest

import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import workloads as W

from gpu_util import check, run_softmax

pytestmark = pytest.mark.gpu
FP32, BF16, FP16 = W.FP32, W.BF16, W.FP16


@pytest.fixture(scope="module", autouse=True)
def status_stays_clean():
    yield
    assert fs.fs_device_status() == fs.FS_OK


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_every_head_offset_and_short_rows(dtype):
    ve = 16 // W.ELEM_SIZE[dtype]
    for cols in (1, 2, 3, 5, 7, 9, 11, 13, 15, 17, 25, 33, 63, 100, 129, 255):
        if (cols * W.ELEM_SIZE[dtype]) % 16 == 0:
            continue
        for rows in (1, 2, ve, 2 * ve + 1, 67, 128, 129, 333, 1025):
            scale = [1.0, 0.5, -1.0][(cols + rows) % 3]
            x = W.random_case(rows, cols, dtype, seed=5000 + cols * 7 + rows, sigma=2.0, neg_inf_frac=0.05 if scale > 0 else 0.0)
            st, y = run_softmax(x, dtype, scale)
            assert st == fs.FS_OK
            check(x, dtype, scale, y)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_row_lengths_up_to_and_beyond_a_block(dtype):
    esz = W.ELEM_SIZE[dtype]
    limit = (128 if dtype == FP32 else 64) * 1024 // esz          # elements a block's registers hold
    for ci, cols in enumerate((1001, 2049, 4099, 8191, 12345, limit - 9, limit - 1, limit + 1, limit + 1001, 50257)):
        if (cols * esz) % 16 == 0:
            cols += 1
        for rows in (1, 5):
            scale = [1.0, 0.25, -0.5][(ci + rows) % 3]
            x = W.random_case(rows, cols, dtype, seed=6000 + ci * 3 + rows, sigma=2.5, neg_inf_frac=0.02 if scale > 0 else 0.0)
            st, y = run_softmax(x, dtype, scale)
            assert st == fs.FS_OK
            check(x, dtype, scale, y)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_in_place_special_values_and_the_element_wise_fallbacks(dtype):
    x = W.random_case(37, 1003, dtype, seed=77, sigma=2.0)
    bits = {FP32: (np.float32(np.nan), np.float32(np.inf), np.float32(-np.inf)),
            BF16: (np.uint16(0x7FC0), np.uint16(0x7F80), np.uint16(0xFF80)),
            FP16: (np.uint16(0x7E00), np.uint16(0x7C00), np.uint16(0xFC00))}[dtype]
    x[1, 0] = bits[0]; x[2, 1002] = bits[1]; x[3, :] = bits[2]; x[4, 1:1000] = bits[2]; x[5, 0] = bits[2]; x[5, 1002] = bits[2]
    for scale in (1.0, -1.0):
        st, y = run_softmax(x, dtype, scale)
        assert st == fs.FS_OK
        check(x, dtype, scale, y)
    st, y = run_softmax(x, dtype, 1.0, inplace=True)                  # neighbours' outputs sit in the shared vectors
    assert st == fs.FS_OK
    check(x, dtype, 1.0, y)
    xs = W.random_case(300, 37, dtype, seed=78, sigma=2.0)             # short rows: spans of 128 rows
    xs[1, 0] = bits[0]; xs[2, 36] = bits[1]; xs[3, :] = bits[2]; xs[130, 1:30] = bits[2]
    for scale, inplace in ((1.0, False), (-1.0, False), (0.0, False), (0.5, True)):
        st, y = run_softmax(xs, dtype, scale, inplace=inplace)
        assert st == fs.FS_OK
        check(xs, dtype, scale, y)
    xl = W.random_case(9, 30011, dtype, seed=79, sigma=2.0)            # long rows: a cluster per row on shifted vectors
    xl[1, 0] = bits[0]; xl[2, 30010] = bits[1]; xl[3, :] = bits[2]; xl[4, 1:30000] = bits[2]; xl[5, 0] = bits[2]; xl[5, 30010] = bits[2]
    for scale, inplace in ((1.0, False), (-1.0, False), (0.0, False), (0.5, True)):
        st, y = run_softmax(xl, dtype, scale, inplace=inplace)
        assert st == fs.FS_OK
        check(xl, dtype, scale, y)
    for kw in (dict(scale=0.0), dict(scale=1.0, offset=1), dict(scale=1.0, threads=64, kernel=fs.FS_KERNEL_GENERIC)):
        scale = kw.pop("scale")                                       # zero scale, unaligned tensors, forced block size
        st, y = run_softmax(x, dtype, scale, **kw)
        assert st == fs.FS_OK
        check(x, dtype, scale, y)


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_many_long_rows(dtype):
    """More rows than resident clusters, every head offset a row can have (the row length is odd)."""
    for rows, cols in ((301, 20001), (130, 50257), (40, 262145)):
        x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.5, neg_inf_frac=0.01)
        st, y = run_softmax(x, dtype, 1.0)
        assert st == fs.FS_OK
        check(x, dtype, 1.0, y)


def test_subnormal_bf16_outputs_survive():
    row = np.linspace(-91.0, -87.0, 1003)
    row[0] = 0.0
    from oracle import fso
    x = fso.round_from_f64(np.tile(row, (3, 1)), BF16)
    st, y = run_softmax(x, BF16, 1.0)
    assert st == fs.FS_OK
    check(x, BF16, 1.0, y)
    assert np.count_nonzero((y[0] > 0) & (y[0] < 0x0080)) > 20
    row = np.linspace(-91.0, -87.0, 30011)                             # the same on the split-row kernel
    row[0] = 0.0
    x = fso.round_from_f64(np.tile(row, (3, 1)), BF16)
    st, y = run_softmax(x, BF16, 1.0)
    assert st == fs.FS_OK
    check(x, BF16, 1.0, y)
    assert np.count_nonzero((y[0] > 0) & (y[0] < 0x0080)) > 500
