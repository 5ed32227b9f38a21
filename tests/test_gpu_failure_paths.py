"""The library's guards, exercised in forms that cannot hurt a device: a bounded wait that is made to run out
(nothing is copied for it, or it is armed for 16 bytes too many: the kernel gives up, finishes and reports), the
per-device scratch buffer of the long-row paths (no allocation per call), and the downgrade paths of a device
without cluster launch or with little shared memory, simulated through the environment in child processes."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fno, fso
from paper_2607_24762_b200 import workloads as W

from gpu_util import check, np_to_torch_bits, run_softmax, torch_bits_to_np

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_a_wait_that_nothing_satisfies_runs_out_and_is_reported_once():
    assert fs.fs_device_status() == fs.FS_OK
    fs.fs_debug_set_wait_polls(64)
    try:
        fs.fs_debug_wait_probe(torch.cuda.current_stream())
        torch.cuda.synchronize()                                    # the kernel returned by itself
        assert fs.fs_device_status() == fs.FS_ERR_DEVICE_TIMEOUT
        assert fs.fs_device_status() == fs.FS_OK                    # cleared by the read
    finally:
        fs.fs_debug_set_wait_polls(0)
    # with the default cap in place an ordinary call is unaffected
    x = W.random_case(8, 16384, W.BF16, seed=3, sigma=2.0)
    status, y = run_softmax(x, W.BF16, 1.0, fs.FS_KERNEL_CLUSTER)
    assert status == fs.FS_OK
    check(x, W.BF16, 1.0, y)
    assert fs.fs_device_status() == fs.FS_OK


@pytest.mark.parametrize("dtype,rows,cols,threads,cluster", [
    (W.BF16, 4, 16384, 0, 1),            # one block per row
    (W.FP32, 6, 32768, 0, 4),            # a cluster of four: the exchange barrier and the exit guard
    (W.BF16, 3, 100000, 0, 0),           # ragged slices, the dispatcher's own geometry
    (W.FP16, 5, 65536, 256, 16),         # sixteen blocks
])
def test_split_row_kernel_gives_up_on_its_waits_and_still_returns(dtype, rows, cols, threads, cluster):
    """Every chunk barrier is armed for 16 bytes more than are copied: each warp's first wait runs out (the
    data itself arrives), the warp stops waiting, the block meets its barriers and the kernel ends."""
    x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.0)
    xd = np_to_torch_bits(x).cuda()
    yd = torch.zeros_like(xd)
    assert fs.fs_device_status() == fs.FS_OK
    fs.fs_debug_set_wait_polls(20000)                               # a few milliseconds: far longer than the copies take
    try:
        st = fs.fs_debug_softmax_expire(xd, yd, rows, cols, dtype, 1.0, torch.cuda.current_stream(), threads, cluster)
        assert st == fs.FS_OK, fs.fs_strerror(st)
        torch.cuda.synchronize()
        assert fs.fs_device_status() == fs.FS_ERR_DEVICE_TIMEOUT
        assert fs.fs_device_status() == fs.FS_OK
    finally:
        fs.fs_debug_set_wait_polls(0)
    if cluster == 1:
        # one block per row depends on no other block: the data had landed, so the result is the normal one
        check(x, dtype, 1.0, torch_bits_to_np(yd, dtype))
    # and the next ordinary launch of the same kernel is clean
    fs.fs_softmax_ex(xd, yd, rows, cols, dtype, 1.0, torch.cuda.current_stream(), fs.FS_KERNEL_CLUSTER, threads, cluster)
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    check(x, dtype, 1.0, torch_bits_to_np(yd, dtype))


def test_long_row_paths_allocate_nothing_after_their_first_call():
    """Rows beyond a cluster's shared memory go through two kernels and a per-device scratch buffer: the second
    call (on another stream) finds the buffer there, free device memory does not move, results stay right."""
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    rows, cols = 3, (1 << 20) + 2048                                # 4 MiB + 8 KiB fp32 rows
    x = W.random_case(rows, cols, W.FP32, seed=9, sigma=2.0, neg_inf_frac=0.01)
    xd = np_to_torch_bits(x).cuda()
    y1, y2 = torch.empty_like(xd), torch.empty_like(xd)
    assert fs.fs_select_kernel(rows, cols, W.FP32) == fs.FS_KERNEL_GENERIC
    gx = fso.round_from_f64(np.random.default_rng(1).standard_normal((2, 1 << 21)) * 1.5 + 0.5, W.BF16)   # 4 MiB bf16 rows
    gxd = np_to_torch_bits(gx).cuda()
    g1, g2 = torch.empty_like(gxd), torch.empty_like(gxd)
    torch.cuda.synchronize()
    with torch.cuda.stream(s1):
        fs.fs_softmax(xd, y1, rows, cols, W.FP32, 1.0, s1)
        fs.fs_layer_norm(gxd, None, None, g1, 2, 1 << 21, W.BF16, 1e-5, s1)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    with torch.cuda.stream(s2):
        fs.fs_softmax(xd, y2, rows, cols, W.FP32, 1.0, s2)
        fs.fs_layer_norm(gxd, None, None, g2, 2, 1 << 21, W.BF16, 1e-5, s2)
    with torch.cuda.stream(s1):                                      # and once more, concurrently, on the first stream
        fs.fs_softmax(xd, y1, rows, cols, W.FP32, 1.0, s1)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert fs.fs_device_status() == fs.FS_OK
    check(x, W.FP32, 1.0, torch_bits_to_np(y1, W.FP32))
    check(x, W.FP32, 1.0, torch_bits_to_np(y2, W.FP32))
    want = fno.layer_norm_f64(gx, W.BF16)
    scale = fno.error_scale(gx, W.BF16, gx.shape)
    for g in (g1, g2):
        assert fno.compare(torch_bits_to_np(g, W.BF16), W.BF16, want, scale).ok(W.BF16)
    fs.fs_release()                                                  # frees the scratch buffer; the next call allocates again
    fs.fs_softmax(xd, y2, rows, cols, W.FP32, 1.0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    check(x, W.FP32, 1.0, torch_bits_to_np(y2, W.FP32))
    fs.fs_release()


_CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, os.path.join(sys.argv[1], "tests"))
import numpy as np, torch
import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import workloads as W
from gpu_util import check, run_softmax
mode = sys.argv[2]
shapes = [(W.BF16, 64, 2048), (W.FP32, 12, 4096), (W.FP32, 9, 16384), (W.BF16, 6, 65536), (W.FP32, 5, 40000), (W.BF16, 3, 262144), (W.FP32, 2, (1 << 20) + 64)]
for dtype, rows, cols in shapes:
    x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.0, neg_inf_frac=0.02)
    status, y = run_softmax(x, dtype, 0.5)                     # the dispatcher's own choice must always run
    assert status == fs.FS_OK, (mode, dtype, rows, cols, fs.fs_strerror(status))
    check(x, dtype, 0.5, y)
    forced, _ = run_softmax(x, dtype, 0.5, fs.FS_KERNEL_CLUSTER, 0, 4)
    if mode == "no_cluster":
        assert forced == fs.FS_ERR_UNSUPPORTED, (dtype, rows, cols, forced)      # a forced geometry is never downgraded
    one, y1 = run_softmax(x, dtype, 0.5, fs.FS_KERNEL_CLUSTER, 0, 1)
    if one == fs.FS_OK:
        check(x, dtype, 0.5, y1)
    elif mode == "small_smem":
        assert one == fs.FS_ERR_UNSUPPORTED
# the other entry points fall back to their generic kernels where the split-row form cannot run
x = W.random_case(4, 65536, W.BF16, seed=5, sigma=2.0)
status, y = run_softmax(x, W.BF16, 1.0, causal_q=65536 - 4)
assert status == fs.FS_OK
from oracle import fso
assert fso.compare(y, W.BF16, fso.softmax_causal_f64(x, W.BF16, 65536 - 4, 1.0)).ok(W.BF16)
assert fs.fs_device_status() == fs.FS_OK
print("downgrade ok", mode)
"""


@pytest.mark.parametrize("mode,env", [("no_cluster", {"FS_SIM_NO_CLUSTER": "1"}), ("small_smem", {"FS_SIM_SMEM_OPTIN": "32768"}),
                                      ("both", {"FS_SIM_NO_CLUSTER": "1", "FS_SIM_SMEM_OPTIN": "32768"})])
def test_downgrade_paths_of_a_lesser_device(mode, env):
    root = os.path.dirname(HERE)
    full = {k: v for k, v in os.environ.items() if not k.startswith("FS_")}
    full.update(env)
    full["FS_LOG"] = "1"
    out = subprocess.run([sys.executable, "-c", _CHILD, root, mode], env=full, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "downgrade ok" in out.stdout
    assert "generic" in out.stderr                                   # FS_LOG shows the dispatcher downgrading
    if "FS_SIM_NO_CLUSTER" in env:
        assert "cluster launch no" in out.stderr


_CHILD_SWITCHES = r"""
import os, sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, os.path.join(sys.argv[1], "tests"))
import numpy as np, torch
import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import workloads as W
from gpu_util import check, run_softmax
x = W.random_case(32, 2048, W.BF16, seed=1, sigma=2.0)
status, y = run_softmax(x, W.BF16, 1.0)
assert status == fs.FS_OK
check(x, W.BF16, 1.0, y)
# FS_CHECK=1: a pageable host pointer is refused before any launch; device tensors pass
host = np.zeros((32, 2048), dtype=np.uint16)
L = fs.binding.lib()
assert L.fs_softmax(host.ctypes.data, host.ctypes.data, 32, 2048, fs.FS_DTYPE_BF16, 1.0, 0) == fs.FS_ERR_INVALID_ARG
# FS_FORCE_KERNEL=block: a row the block kernel cannot hold is refused, not rerouted
xl = W.random_case(4, 65536, W.BF16, seed=2, sigma=2.0)
status, _ = run_softmax(xl, W.BF16, 1.0)
assert status == fs.FS_ERR_UNSUPPORTED, status
torch.cuda.synchronize()
assert fs.fs_device_status() == fs.FS_OK
print("switches ok")
"""


def test_log_force_and_check_switches():
    root = os.path.dirname(HERE)
    full = {k: v for k, v in os.environ.items() if not k.startswith("FS_")}
    full.update({"FS_LOG": "1", "FS_FORCE_KERNEL": "block", "FS_CHECK": "1"})
    out = subprocess.run([sys.executable, "-c", _CHILD_SWITCHES, root], env=full, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "switches ok" in out.stdout
    assert "[fsoftmax] softmax 32 x 2048 dtype 1: block kernel" in out.stderr
    assert "FS_CHECK" in out.stderr
