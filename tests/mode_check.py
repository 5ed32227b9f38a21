"""Parity sweep used by test_gpu_modes.py in a child process (the library reads its environment
switches once per process): every kernel on a handful of shapes, all dtypes, against the oracle."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np  # noqa: E402

import paper_2607_24762_b200 as fs  # noqa: E402
from paper_2607_24762_b200 import workloads as W  # noqa: E402

from gpu_util import check, run_softmax  # noqa: E402


def main() -> int:
    ran = 0
    shapes = [(1, 8), (300, 128), (2000, 256), (77, 1000), (600, 2048), (513, 4096), (129, 16384), (70, 40000),
              (37, 65536), (9, 262144), (5, 100000), (130, 37), (21, 1001), (3, 50257)]
    for dtype in (W.FP32, W.BF16, W.FP16):
        for rows, cols in shapes:
            x = W.random_case(rows, cols, dtype, seed=rows + cols, sigma=2.5, neg_inf_frac=0.03)
            for kernel in range(0, 6):
                for scale in (1.0, -0.5):
                    xs = x if scale > 0 else W.random_case(rows, cols, dtype, seed=rows + cols + 1, sigma=2.5)
                    status, y = run_softmax(xs, dtype, scale, kernel)
                    if status == fs.FS_ERR_UNSUPPORTED and kernel != fs.FS_KERNEL_AUTO:
                        continue
                    assert status == fs.FS_OK, (rows, cols, dtype, kernel, fs.fs_strerror(status), fs.fs_last_cuda_error())
                    check(xs, dtype, scale, y)
                    ran += 1
    # many rows per launch: several generations of resident blocks
    for dtype, rows, cols in ((W.BF16, 40000, 512), (W.FP32, 6000, 8192), (W.BF16, 3000, 32768)):
        x = W.random_case(rows, cols, dtype, seed=5, sigma=2.0, neg_inf_frac=0.01)
        for kernel in (fs.FS_KERNEL_WARP, fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA, fs.FS_KERNEL_CLUSTER):
            status, y = run_softmax(x, dtype, 1.0, kernel)
            if status == fs.FS_ERR_UNSUPPORTED:
                continue
            assert status == fs.FS_OK
            step = max(1, (1 << 22) // cols)
            for r0 in range(0, rows, step):
                check(x[r0:r0 + step], dtype, 1.0, y[r0:r0 + step])
            ran += 1
    assert fs.fs_device_status() == fs.FS_OK
    print(f"mode_check ok: {ran} cases, env " +
          " ".join(f"{k}={v}" for k, v in sorted(os.environ.items()) if k.startswith("FS_")))
    return 0


if __name__ == "__main__":
    sys.exit(main())
