"""GPU parity of fs_softmax_backward against the fp64 oracle, element by element on seeded inputs,
through the C ABI. The bar: fp32 |error| <= 2e-6 x the element's error scale |scale| |y| (|dy| + sum
|dy y|) (the products and the row sum are binary32); bf16/fp16 within one unit in the last place of
the correctly rounded fp64 value, or within that bound where dy and the dot product cancel."""
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


def make(rows, cols, dtype, seed):
    """y: a softmax output rounded to dtype (through the oracle); dy: seeded normal values."""
    x = W.random_case(rows, cols, dtype, seed=seed, sigma=2.0, neg_inf_frac=0.02)
    y = fso.round_from_f64(fso.softmax_f64(x, dtype, 1.0), dtype)
    dy = fso.round_from_f64(np.random.default_rng(seed + 1).standard_normal((rows, cols)), dtype)
    return dy, y


def run(dy, y, dtype, scale, alias=None, misalign=0):
    rows, cols = y.shape
    pad = lambda a: np.concatenate([np.zeros(misalign, a.dtype), a.ravel()])
    gd, yd = np_to_torch_bits(pad(dy)).cuda(), np_to_torch_bits(pad(y)).cuda()
    dd = gd if alias == "dy" else yd if alias == "y" else torch.zeros_like(gd)
    off = misalign * W.ELEM_SIZE[dtype]
    fs.fs_softmax_backward(gd.data_ptr() + off, yd.data_ptr() + off, dd.data_ptr() + off, rows, cols, dtype, scale,
                           torch.cuda.current_stream())
    torch.cuda.synchronize()
    return torch_bits_to_np(dd, dtype)[misalign:].reshape(rows, cols)


def check(dy, y, dtype, scale, **kw):
    got = run(dy, y, dtype, scale, **kw)
    want = fso.softmax_backward_f64(dy, y, dtype, scale)
    err_scale = fno.backward_error_scale(dy, y, dtype, scale)      # pinned in tests/test_oracle_backward_pins.py
    rep = fno.compare(got, dtype, want, np.where(np.isfinite(err_scale), err_scale, 1.0))
    assert rep.ok(dtype), (y.shape, dtype, scale, rep)
    return rep


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_shape_sweep(dtype):
    scales = [1.0, 0.5, 128 ** -0.5, -1.0, 0.0]
    for ci, cols in enumerate([1, 2, 3, 8, 16, 17, 100, 128, 257, 512, 1000, 1024, 1536, 2048, 4096, 5000, 8192, 16384, 40000,
                               65536, 100000, 262144, 300001]):
        for rows in ((1, 3, 65) if cols <= 16384 else (1, 5)):
            dy, y = make(rows, cols, dtype, seed=500 + ci)
            check(dy, y, dtype, scales[(ci + rows) % len(scales)])


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_row_lengths_across_the_split_geometries(dtype):
    esz = W.ELEM_SIZE[dtype]
    for kb, rows in ((3, 700), (8, 2000), (12, 900), (24, 400), (40, 300), (96, 150), (100, 120), (160, 100), (250.5, 60), (384, 40),
                     (512, 200), (600, 30), (1024, 12), (2048, 5)):
        cols = int(kb * 1024) // esz
        dy, y = make(rows, cols, dtype, seed=int(kb))
        check(dy, y, dtype, 0.25)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_rows_around_the_four_rows_per_block_kernel(dtype):
    """Rows of 257..512 sixteen-byte vectors take the kernel that works on four row pairs per block from
    shared memory: both ends of that range and one vector beyond them, row counts that leave a block
    partly empty, dx aliasing dy or y."""
    ve = 16 // W.ELEM_SIZE[dtype]
    for ci, nvec in enumerate((256, 257, 300, 511, 512, 513)):
        for rows in (1, 4, 5, 7, 130):
            dy, y = make(rows, nvec * ve, dtype, seed=40 * nvec + rows)
            check(dy, y, dtype, [1.0, 0.25, -0.5][(ci + rows) % 3], alias=[None, "dy", "y"][(ci + rows) % 3])


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_aliasing_alignment_and_special_values(dtype):
    dy, y = make(33, 2048, dtype, seed=3)
    check(dy, y, dtype, 1.0, alias="dy")
    check(dy, y, dtype, 1.0, alias="y")
    dy, y = make(5, 65536, dtype, seed=4)
    check(dy, y, dtype, 1.0, alias="dy")
    dy, y = make(9, 1001, dtype, seed=5)
    check(dy, y, dtype, 0.7)                                  # ragged columns: generic kernel
    dy, y = make(9, 1024, dtype, seed=6)
    check(dy, y, dtype, 0.7, misalign=1)
    dy, y = make(6, 4096, dtype, seed=7)
    dy[2, 100] = np.float32(np.nan) if dtype == FP32 else np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    check(dy, y, dtype, 1.0)                                  # a NaN gradient poisons its row only
    fs.fs_softmax_backward(None, None, None, 0, 128, dtype)
    L = fs.binding.lib()
    a, b = 0x10000, 0x2000000
    assert L.fs_softmax_backward(a, a + 0x100000, b, -1, 8, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG
    assert L.fs_softmax_backward(a, a + 0x100000, a + 16, 8, 8, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG
    assert L.fs_softmax_backward(None, a, b, 8, 8, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG


def test_attention_workload_full_size():
    """cfg2's attention-score shape (16384 x 2048 bf16): the softmax output and a seeded gradient."""
    w = W.WORKLOADS["cfg2"]
    x = W.generate_rows(w, 0, w.rows)
    y = fso.round_from_f64(fso.softmax_f64(x, w.dtype, w.scale_f32), w.dtype)
    dy = fso.round_from_f64(np.random.default_rng(77).standard_normal((w.rows, w.cols)), w.dtype)
    rep = check(dy, y, w.dtype, w.scale_f32)
    print("cfg2 backward", rep)
