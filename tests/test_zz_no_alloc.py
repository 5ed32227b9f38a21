"""fs_softmax_static: the entry point for callers that must never allocate device memory (a process
whose memory pool owns the whole GPU, a service that must not be able to run out of memory after
start-up, a loop that cannot take the allocator's device synchronisation). What the other entry
points keep in cudaMalloc'ed memory -- the status buffer of the bounded waits, and the per-segment
(max, sum) pairs that the two kernels of the long-row path hand to each other -- lives in a fixed
64 KiB device array instead. The checks: same bits as the existing entry point running the same
kernels, on two calls in a row (the array is shared and keeps the previous call's contents), plus
the oracle's tolerance; a clear refusal of what it does not take; a readable status word; and, in a
fresh process, free device memory that does not move across its calls.

Collected last on purpose: if this file fails, a run that stops at the first failure has already
run every other test. It passes on its own in a fresh process as well."""
import os
import subprocess
import sys

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


def test_static_long_rows_use_the_fixed_array_twice():
    """Rows beyond a cluster's shared memory: two kernels, the pairs between them in the fixed array.
    Same bits as fs_softmax, whose dispatcher runs the same two kernels with the pairs in its own buffer."""
    for dtype, rows, cols, scale in ((W.FP32, 3, (1 << 20) + 4096, 1.0), (W.BF16, 5, (1 << 21) + 64, -0.5)):
        assert cols * W.ELEM_SIZE[dtype] > fs.FS_STATIC_MAX_ROW_BYTES
        x = W.random_case(rows, cols, dtype, seed=cols, sigma=2.5, neg_inf_frac=0.01 if scale > 0 else 0.0)
        xd = np_to_torch_bits(x).cuda()
        stream = torch.cuda.current_stream()
        ref = torch.empty_like(xd)
        fs.fs_softmax(xd, ref, rows, cols, dtype, scale, stream)
        torch.cuda.synchronize()
        for call in range(2):
            got = torch.full_like(xd, 0x7FC0 if dtype != W.FP32 else float("nan"))
            fs.fs_softmax_static(xd, got, rows, cols, dtype, scale, stream)
            torch.cuda.synchronize()
            assert torch.equal(got.view(torch.uint8), ref.view(torch.uint8)), f"call {call} differs"
        check(x, dtype, scale, torch_bits_to_np(got, dtype))
        assert fs.fs_static_status() == fs.FS_OK


def test_static_entry_point_refuses_what_it_cannot_take():
    L = fs.binding.lib()
    a = torch.zeros(1 << 22, dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    s = torch.cuda.current_stream().cuda_stream
    big_cols = fs.FS_STATIC_MAX_ROW_BYTES // 4 + 4                                   # one vector past the split-row kernel's limit
    # more (row, segment) pairs than the fixed array holds: refused before anything is enqueued or touched
    many = fs.FS_STATIC_MAX_PAIRS + 1
    assert L.fs_softmax_static(a.data_ptr(), a.data_ptr(), many, big_cols, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(a.data_ptr(), b.data_ptr(), 8, 1023, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(a.data_ptr() + 4, b.data_ptr(), 8, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_UNSUPPORTED
    assert L.fs_softmax_static(0, b.data_ptr(), 8, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_ERR_INVALID_ARG
    assert L.fs_softmax_static(a.data_ptr(), b.data_ptr(), 0, 1024, fs.FS_DTYPE_FP32, 1.0, s) == fs.FS_OK
    assert "unsupported" in fs.fs_strerror(fs.FS_ERR_UNSUPPORTED)
    torch.cuda.synchronize()
    # the largest row the split-row kernel takes
    cols = fs.FS_STATIC_MAX_ROW_BYTES // 4
    x = W.random_case(1, cols, W.FP32, seed=4, sigma=2.0)
    xd = np_to_torch_bits(x).cuda()
    yd = torch.empty_like(xd)
    fs.fs_softmax_static(xd, yd, 1, cols, W.FP32, 1.0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    check(x, W.FP32, 1.0, torch_bits_to_np(yd, W.FP32))
    assert fs.fs_static_status() == fs.FS_OK


_CHILD = r"""
import sys
sys.path.insert(0, sys.argv[1])
import torch
import paper_2607_24762_b200 as fs
torch.cuda.set_device(0)
stream = torch.cuda.current_stream()
cases = [(fs.FS_DTYPE_BF16, 16, 262144), (fs.FS_DTYPE_FP32, 2, (1 << 20) + 4096)]      # split-row kernel; long-row path
bufs = [(torch.randn(r, c, device="cuda").to(torch.bfloat16 if d == fs.FS_DTYPE_BF16 else torch.float32), d, r, c) for d, r, c in cases]
outs = [torch.empty_like(b[0]) for b in bufs]
assert fs.fs_static_status() == fs.FS_OK          # loads the library's device code (module loading is set to eager)
torch.cuda.synchronize()
free = [torch.cuda.mem_get_info()[0]]
for call in range(2):
    for (x, d, r, c), y in zip(bufs, outs):
        fs.fs_softmax_static(x, y, r, c, d, 1.0, stream)
    torch.cuda.synchronize()
    free.append(torch.cuda.mem_get_info()[0])
assert fs.fs_static_status() == fs.FS_OK
for (x, d, r, c), y in zip(bufs, outs):
    assert torch.allclose(y.float().sum(dim=1), torch.ones(r, device="cuda"), atol=2e-2)
print("FREE", *free)
"""


def test_static_entry_point_leaves_free_device_memory_alone():
    """A fresh process in which no other entry point of the library has run: free device memory, as the
    driver reports it, is the same before the first call, after it and after the second (the library's
    code is loaded up front, so that lazy loading of kernels does not blur the reading)."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, CUDA_MODULE_LOADING="EAGER")
    out = subprocess.run([sys.executable, "-c", _CHILD, root], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    free = [int(v) for v in out.stdout.split("FREE")[1].split()]
    assert len(free) == 3 and free[0] == free[1] == free[2], free
