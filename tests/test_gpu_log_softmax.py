"""GPU parity of fs_log_softmax against the fp64 oracle, element by element on seeded inputs, through
the C ABI. The bar: fp32 |error| <= 1e-6 * max(1, |y|); bf16/fp16 within one unit in the last place of
the correctly rounded fp64 value (or that fp32 bound); -inf and NaN where the oracle has them."""
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


def run(x, dtype, scale, misalign=0, inplace=False):
    rows, cols = x.shape
    xd = np_to_torch_bits(np.concatenate([np.zeros(misalign, x.dtype), x.ravel()])).cuda()
    yd = xd if inplace else torch.zeros_like(xd)
    esz = W.ELEM_SIZE[dtype]
    fs.fs_log_softmax(xd.data_ptr() + misalign * esz, yd.data_ptr() + misalign * esz, rows, cols, dtype, scale,
                      torch.cuda.current_stream())
    torch.cuda.synchronize()
    return torch_bits_to_np(yd, dtype)[misalign:].reshape(rows, cols)


def check(x, dtype, scale, **kw):
    y = run(x, dtype, scale, **kw)
    want = fso.log_softmax_f64(x, dtype, scale)
    rep = fno.compare(y, dtype, want, fno.log_softmax_bound(want), rel_tol=1.0)      # the bound is pinned in tests/test_oracle_log_softmax_pins.py
    assert rep.ok(dtype, rel_tol=1.0), (x.shape, dtype, scale, rep)
    # -inf exactly where the oracle has it
    g64 = fso.widen(y, dtype)
    assert np.array_equal(np.isneginf(g64), np.isneginf(want))
    return rep


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_shape_sweep(dtype):
    scales = [1.0, 0.5, 128 ** -0.5, -1.0, 0.0, 3.0]
    for ci, cols in enumerate([1, 2, 3, 8, 16, 17, 100, 128, 257, 512, 1000, 1024, 1536, 2048, 4096, 5000, 8192, 12288, 16384,
                               40000, 65536, 100000, 262144, 300001]):
        for rows in ((1, 3, 65) if cols <= 16384 else (1, 5)):
            scale = scales[(ci + rows) % len(scales)]
            x = W.random_case(rows, cols, dtype, seed=300 + ci, sigma=3.0, neg_inf_frac=0.03 if scale > 0 else 0.0)
            check(x, dtype, scale)


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_row_lengths_across_the_split_geometries(dtype):
    esz = W.ELEM_SIZE[dtype]
    for kb, rows in ((6, 500), (8, 3000), (12, 900), (24, 400), (40, 300), (48, 260), (96, 150), (100, 120), (160, 100), (250.5, 60),
                     (384, 40), (512, 300), (600, 30), (1024, 12), (2048, 5), (4096, 2)):
        cols = int(kb * 1024) // esz
        x = W.random_case(rows, cols, dtype, seed=int(kb), sigma=4.0)
        check(x, dtype, 1.0 if int(kb) % 2 else -0.5)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_rows_around_the_four_rows_per_block_kernel(dtype):
    """Rows of 257..768 sixteen-byte vectors take the kernel that works on four rows per block from shared
    memory: both ends of that range and one vector beyond them, row counts that leave a block partly
    empty, positive, negative and zero scale, in place."""
    ve = 16 // W.ELEM_SIZE[dtype]
    for ci, nvec in enumerate((256, 257, 400, 767, 768, 769)):
        for rows in (1, 4, 5, 7, 130):
            scale = [1.0, 0.25, -0.5, 0.0][(ci + rows) % 4]
            x = W.random_case(rows, nvec * ve, dtype, seed=50 * nvec + rows, sigma=2.0, neg_inf_frac=0.03 if scale > 0 else 0.0)
            check(x, dtype, scale, inplace=(rows == 5))


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_special_values_alignment_and_aliasing(dtype):
    x = W.random_case(6, 4096, dtype, seed=5, sigma=2.0)
    nan_bits = np.float32(np.nan) if dtype == FP32 else np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    pinf = np.float32(np.inf) if dtype == FP32 else np.uint16(0x7F80 if dtype == BF16 else 0x7C00)
    ninf = np.float32(-np.inf) if dtype == FP32 else np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    x[1, 7] = nan_bits
    x[2, 4000] = pinf
    x[3, :] = ninf
    x[4, 100:200] = ninf
    for scale in (1.0, -1.0, 0.0):
        check(x, dtype, scale)
    check(W.random_case(9, 1001, dtype, seed=6, sigma=2.0), dtype, 0.7)               # ragged columns: generic kernel
    check(W.random_case(9, 1024, dtype, seed=7, sigma=2.0), dtype, 0.7, misalign=1)  # misaligned base
    check(W.random_case(33, 2048, dtype, seed=8, sigma=2.0), dtype, 1.0, inplace=True)
    check(W.random_case(5, 65536, dtype, seed=9, sigma=2.0), dtype, 1.0, inplace=True)
    fs.fs_log_softmax(None, None, 0, 128, dtype)
    fs.fs_log_softmax(None, None, 128, 0, dtype)


def test_vocabulary_workload_full_size():
    """cfg4's vocabulary-sized rows (256 x 262144 bf16, spikes at +30): the shape log_softmax is used on."""
    w = W.WORKLOADS["cfg4"]
    x = W.generate_rows(w, 0, w.rows)
    rep = check(x, w.dtype, w.scale_f32)
    print("cfg4 log_softmax", rep)


def test_rejects_bad_arguments():
    a, b = 0x10000, 0x2000000
    L = fs.binding.lib()
    bad = fs.FS_ERR_INVALID_ARG
    assert L.fs_log_softmax(a, b, -1, 8, FP32, 1.0, None) == bad
    assert L.fs_log_softmax(a, b, 8, 8, 9, 1.0, None) == bad
    assert L.fs_log_softmax(a, b, 8, 8, FP32, float("inf"), None) == bad
    assert L.fs_log_softmax(None, b, 8, 8, FP32, 1.0, None) == bad
    assert L.fs_log_softmax(a, a + 16, 8, 8, FP32, 1.0, None) == bad
