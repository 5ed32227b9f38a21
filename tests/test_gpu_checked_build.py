"""The checked build of the library (libfsoftmax_debug.so, -DFS_DEBUG_BOUNDS): every global access of every
kernel is compared with the address ranges of the call's tensors, and an access outside them is skipped and
reported instead of performed. Two things are shown, in a child process that loads that build: correct kernels
raise no report on any entry point (and still meet the oracle), and a kernel that runs past its output --
simulated by registering an output range that ends 4 KiB early, so that nothing is really overrun -- is caught:
status FS_ERR_DEVICE_BOUNDS, the first refused address inside the cut-off tail, the tail left untouched."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, os.path.join(sys.argv[1], "tests"))
import numpy as np, torch
import paper_2607_24762_b200 as fs
from oracle import fno, fso
from paper_2607_24762_b200 import workloads as W
from gpu_util import check, np_to_torch_bits, run_softmax, torch_bits_to_np
assert fs.fs_debug_checked_build() and "checked" in fs.fs_version()
S = torch.cuda.current_stream()
ran = 0
# every softmax kernel, aligned and misaligned, ragged and whole slices
for dtype, rows, cols in ((W.BF16, 300, 128), (W.FP32, 64, 1000), (W.BF16, 70, 2048), (W.FP16, 33, 4096), (W.FP32, 9, 16384),
                          (W.BF16, 5, 100000), (W.BF16, 3, 262144), (W.FP32, 2, (1 << 20) + 64), (W.FP16, 7, 1001)):
    x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.0, neg_inf_frac=0.02)
    for kernel in range(6):
        for offset in (0, 1):
            status, y = run_softmax(x, dtype, 0.5, kernel, offset=offset)
            if status == fs.FS_ERR_UNSUPPORTED and kernel != fs.FS_KERNEL_AUTO:
                continue
            assert status == fs.FS_OK, (dtype, rows, cols, kernel, offset, status)
            check(x, dtype, 0.5, y)
            assert fs.fs_device_status() == fs.FS_OK, ("false report", dtype, rows, cols, kernel, offset, hex(fs.fs_debug_bad_address()))
            ran += 1
# the other entry points, once each on a fast and on a generic shape
def dev(a, dtype):
    return np_to_torch_bits(a).cuda()
for dtype, rows, cols in ((W.BF16, 48, 2048), (W.FP32, 6, 40960), (W.FP16, 5, 1001)):
    x = W.random_case(rows, cols, dtype, seed=3, sigma=2.0)
    xd = dev(x, dtype); yd = torch.empty_like(xd)
    fs.fs_softmax_causal(xd, yd, rows, cols, cols - rows, dtype, 0.5, S)
    fs.fs_log_softmax(xd, yd, rows, cols, dtype, 1.0, S)
    fs.fs_softmax(xd, yd, rows, cols, dtype, 1.0, S)
    gd = dev(fso.round_from_f64(np.random.default_rng(1).standard_normal((rows, cols)), dtype), dtype)
    dd = torch.empty_like(xd)
    fs.fs_softmax_backward(gd, yd, dd, rows, cols, dtype, 1.0, S)
    md = dev(fso.round_from_f64(np.zeros((rows // 1, cols)), dtype), dtype)
    fs.fs_softmax_masked(xd, md, yd, rows, cols, rows, 1, dtype, 1.0, S)
    wd = dev(fso.round_from_f64(np.ones(cols), dtype), dtype)
    fs.fs_layer_norm(xd, wd, None, yd, rows, cols, dtype, 1e-5, S)
    if cols % 8 == 0:
        fs.fs_group_norm(xd, None, None, yd, 1, rows, cols, rows // 2 if rows % 2 == 0 else 1, dtype, 1e-5, S)
    if dtype != W.FP32:
        fo = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
        fs.fs_softmax_f32out(xd, fo, rows, cols, dtype, 1.0, S)
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK, ("false report", dtype, rows, cols, hex(fs.fs_debug_bad_address()))
    ran += 1
x = W.random_case(512, 128, W.BF16, seed=13, sigma=1.0)
xd = dev(x, W.BF16)
wd = torch.empty((512, 8), dtype=torch.float32, device="cuda"); idd = torch.empty((512, 8), dtype=torch.int32, device="cuda")
fs.fs_router_topk(xd, wd, idd, 512, 128, 8, W.BF16, 1.0, True, S)
fs.fs_copy(xd, torch.empty_like(xd), 512 * 128 * 2, S)
torch.cuda.synchronize()
assert fs.fs_device_status() == fs.FS_OK and fs.fs_debug_bad_address() == 0

# a kernel that "runs past" its output: the registered output range ends 4096 bytes early
cut = 4096
for dtype, rows, cols, kernel in ((W.BF16, 64, 2048, fs.FS_KERNEL_WARP), (W.FP32, 64, 2048, fs.FS_KERNEL_BLOCK), (W.BF16, 8, 65536, fs.FS_KERNEL_CLUSTER),
                                  (W.FP16, 9, 1001, fs.FS_KERNEL_GENERIC)):
    x = W.random_case(rows, cols, dtype, seed=7, sigma=2.0)
    xd = dev(x, dtype)
    yd = torch.full_like(xd, 0x5A5A if dtype != W.FP32 else 1234.5)
    nbytes = rows * cols * W.ELEM_SIZE[dtype]
    fs.fs_debug_shrink_writable(cut)
    try:
        fs.fs_softmax_ex(xd, yd, rows, cols, dtype, 1.0, S, kernel)
        torch.cuda.synchronize()
    finally:
        fs.fs_debug_shrink_writable(0)
    assert fs.fs_device_status() == fs.FS_ERR_DEVICE_BOUNDS
    assert fs.fs_device_status() == fs.FS_OK
    bad = fs.fs_debug_bad_address()
    assert yd.data_ptr() + nbytes - cut <= bad < yd.data_ptr() + nbytes, (hex(bad), hex(yd.data_ptr()), nbytes)
    assert fs.fs_debug_bad_address() == 0
    raw = yd.view(torch.uint8).flatten()
    tail = raw[nbytes - cut + 16:]                                   # a 16-byte vector may straddle the cut: it is refused whole
    fill = torch.full_like(xd, 0x5A5A if dtype != W.FP32 else 1234.5).view(torch.uint8).flatten()[nbytes - cut + 16:]
    assert torch.equal(tail, fill), "the checker let a store through"
    head_rows = (nbytes - cut) // (cols * W.ELEM_SIZE[dtype]) - 1     # rows wholly before the cut are complete and right
    if head_rows > 0:
        check(x[:head_rows], dtype, 1.0, torch_bits_to_np(yd, dtype)[:head_rows])
    ran += 1
print("checked build ok", ran)
"""


def test_checked_build_reports_nothing_on_correct_kernels_and_catches_an_overrun():
    sys.path.insert(0, ROOT)
    from paper_2607_24762_b200 import _build
    lib = _build.build_library(debug=True)
    env = {k: v for k, v in os.environ.items() if not k.startswith("FS_")}
    env["FSOFTMAX_LIB"] = lib
    out = subprocess.run([sys.executable, "-c", _CHILD, ROOT], env=env, capture_output=True, text=True, timeout=1800)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "checked build ok" in out.stdout
