"""GPU parity of fs_softmax_f32out (bf16/fp16 in, float32 out) against the fp64 softmax oracle on the
same stored inputs: every output within 1e-6 of the fp64 value, exact +0 for -inf entries, NaN rows
where the oracle has them."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fso
from paper_2607_24762_b200 import workloads as W
from tests.gpu_util import np_to_torch_bits

pytestmark = pytest.mark.gpu
BF16, FP16, FP32 = W.BF16, W.FP16, W.FP32


@pytest.fixture(scope="module", autouse=True)
def built_library():
    from paper_2607_24762_b200 import _build
    _build.build_library()
    yield
    assert fs.fs_device_status() == fs.FS_OK


def check(x, dtype, scale, misalign=0, y_offset=0):
    """y_offset: floats in front of y (0: 32-byte aligned, one 256-bit store per vector; 4: 16-byte aligned, two
    128-bit stores; 1: element-wise kernel)."""
    rows, cols = x.shape
    xd = np_to_torch_bits(np.concatenate([np.zeros(misalign, x.dtype), x.ravel()])).cuda()
    yd = torch.full((y_offset + rows * cols + 8,), 7.0, dtype=torch.float32, device="cuda")  # guard floats in front and behind
    fs.binding._check(fs.binding.lib().fs_softmax_f32out(xd.data_ptr() + 2 * misalign, yd.data_ptr() + 4 * y_offset, rows, cols, dtype,
                                                        scale, torch.cuda.current_stream().cuda_stream), "fs_softmax_f32out")
    torch.cuda.synchronize()
    got = yd.cpu().numpy()
    assert np.all(got[:y_offset] == 7.0) and np.all(got[y_offset + rows * cols:] == 7.0)
    got = got[y_offset:]
    rep = fso.compare(got[:rows * cols].reshape(rows, cols), FP32, fso.softmax_f64(x, dtype, scale))
    assert rep.ok(FP32), (x.shape, dtype, scale, rep)
    return rep


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_shape_sweep(dtype):
    scales = [1.0, 0.5, 128 ** -0.5, -1.0, 0.0]
    for ci, cols in enumerate([1, 2, 3, 8, 16, 17, 100, 128, 257, 512, 1000, 1024, 1536, 2048, 3072, 4096, 5000, 8192, 16384, 40000,
                               65536, 100000, 262144, 300008, (1 << 21) + 8]):
        for rows in ((1, 3, 65) if cols <= 16384 else (1, 4)):
            scale = scales[(ci + rows) % len(scales)]
            x = W.random_case(rows, cols, dtype, seed=700 + ci, sigma=2.5, neg_inf_frac=0.03 if scale > 0 else 0.0)
            check(x, dtype, scale)


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_rows_around_the_four_rows_per_block_kernel(dtype):
    """Rows of 257..768 sixteen-byte vectors take the kernel that works on four rows per block from shared
    memory: both ends of that range, one vector beyond them, row counts that leave a block partly empty."""
    for ci, nvec in enumerate((256, 257, 400, 767, 768, 769)):
        for rows in (1, 4, 5, 7, 130):
            scale = [1.0, 0.25, -0.5, 0.0][(ci + rows) % 4]
            x = W.random_case(rows, nvec * 8, dtype, seed=60 * nvec + rows, sigma=2.0, neg_inf_frac=0.03 if scale > 0 else 0.0)
            check(x, dtype, scale)


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_output_alignments(dtype):
    """y at a 32-byte boundary leaves in 256-bit stores, at a 16-byte boundary in pairs of 128-bit stores, anywhere
    else through the element-wise kernel: the warp kernel, the four-rows-per-block kernel and the split-row kernel."""
    for ci, (rows, cols) in enumerate(((67, 2048), (9, 3072), (5, 65536), (3, 100000))):
        x = W.random_case(rows, cols, dtype, seed=4100 + ci, sigma=2.0, neg_inf_frac=0.02)
        for y_offset in (0, 4, 8, 12, 1):
            check(x, dtype, [1.0, 0.5][ci % 2], y_offset=y_offset)


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_special_values_alignment_and_workload(dtype):
    x = W.random_case(6, 4096, dtype, seed=5, sigma=2.0)
    x[1, 7] = np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    x[2, 4000] = np.uint16(0x7F80 if dtype == BF16 else 0x7C00)
    x[3, :] = np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    x[4, 100:200] = np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    for scale in (1.0, -1.0, 0.0):
        check(x, dtype, scale)
    check(W.random_case(9, 1024, dtype, seed=7, sigma=2.0), dtype, 0.7, misalign=1)          # misaligned input: generic kernel
    fs.fs_softmax_f32out(None, None, 0, 128, dtype)
    L = fs.binding.lib()
    a, b = 0x10000, 0x2000000
    assert L.fs_softmax_f32out(a, b, 8, 8, FP32, 1.0, None) == fs.FS_ERR_INVALID_ARG       # 16-bit inputs only
    assert L.fs_softmax_f32out(a, a + 64, 8, 8, dtype, 1.0, None) == fs.FS_ERR_INVALID_ARG  # overlap
    assert L.fs_softmax_f32out(a, b, 8, 8, dtype, float("nan"), None) == fs.FS_ERR_INVALID_ARG


def test_attention_workload_full_size():
    w = W.WORKLOADS["cfg2"]
    rep = check(W.generate_rows(w, 0, w.rows), w.dtype, w.scale_f32)
    print("cfg2 f32out", rep)
