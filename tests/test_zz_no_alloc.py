"""fs_softmax_static: the entry point for callers that must never allocate device memory (a process
whose memory pool owns the whole GPU, a service that must not be able to run out of memory after
start-up, a loop that cannot take the allocator's device synchronisation). It runs the split-row
kernel with the kernel's status word in a fixed 256-byte device array instead of a cudaMalloc'ed
buffer. The check: same bits as the existing entry point running the same kernel, on two calls in a
row (the array is shared and keeps the previous call's contents), plus the oracle's tolerance, and a
clear refusal of what it does not take.

Collected last on purpose: if this file fails, a run that stops at the first failure has already
run every other test. It passes on its own in a fresh process as well."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import workloads as W

from gpu_util import check, np_to_torch_bits, torch_bits_to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,rows,cols,scale", [
    (W.BF16, 24, 262144, 1.0),          # vocabulary-sized rows: 16 blocks per row
    (W.FP32, 70, 40000, 0.5),           # 160 KB rows: a ragged last slice
    (W.FP16, 300, 2048, -1.0),          # one block per row, negative scale
])
def test_static_entry_point_matches_the_allocating_one_twice(dtype, rows, cols, scale):
    from paper_2607_24762_b200 import _build
    _build.build_library()
    x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.5, neg_inf_frac=0.02 if scale > 0 else 0.0)
    xd = np_to_torch_bits(x).cuda()
    stream = torch.cuda.current_stream()
    ref = torch.empty_like(xd)
    fs.fs_softmax_ex(xd, ref, rows, cols, dtype, scale, stream, fs.FS_KERNEL_CLUSTER)
    torch.cuda.synchronize()
    for call in range(2):
        got = torch.full_like(xd, 0x7FC0 if dtype != W.FP32 else float("nan"))
        fs.fs_softmax_static(xd, got, rows, cols, dtype, scale, stream)
        torch.cuda.synchronize()
        assert torch.equal(got.view(torch.uint8), ref.view(torch.uint8)), f"call {call} differs"
    check(x, dtype, scale, torch_bits_to_np(got, dtype))
    # in place, on a side stream
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    buf = xd.clone()
    fs.fs_softmax_static(buf, buf, rows, cols, dtype, scale, side)
    side.synchronize()
    assert torch.equal(buf.view(torch.uint8), ref.view(torch.uint8))


def test_static_entry_point_refuses_what_it_cannot_take():
    L = fs.binding.lib()
    a = torch.zeros(1 << 22, dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    s = torch.cuda.current_stream().cuda_stream
    big_cols = fs.FS_STATIC_MAX_ROW_BYTES // 4 + 4                                   # one vector past the limit
    assert L.fs_softmax_static(a.data_ptr(), b.data_ptr(), 1, big_cols, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(a.data_ptr(), b.data_ptr(), 8, 1023, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(a.data_ptr() + 4, b.data_ptr(), 8, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(0, b.data_ptr(), 8, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_INVALID_ARG
    assert L.fs_softmax_static(a.data_ptr(), b.data_ptr(), 0, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_OK
    assert "unsupported" in fs.fs_strerror(fs.FS_ERR_UNSUPPORTED)
    torch.cuda.synchronize()
    # the largest row it does take
    cols = fs.FS_STATIC_MAX_ROW_BYTES // 4
    x = W.random_case(1, cols, W.FP32, seed=4, sigma=2.0)
    xd = np_to_torch_bits(x).cuda()
    yd = torch.empty_like(xd)
    fs.fs_softmax_static(xd, yd, 1, cols, W.FP32, 1.0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    check(x, W.FP32, 1.0, torch_bits_to_np(yd, W.FP32))
