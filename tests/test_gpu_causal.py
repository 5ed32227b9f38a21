"""GPU parity of fs_softmax_causal (row i keeps columns j <= i + q_offset) against the oracle's
causal softmax, under the same bar as the plain softmax. Masked inputs hold garbage (NaN, inf,
huge values) on purpose: they must not be looked at."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fso
from paper_2607_24762_b200 import workloads as W

from gpu_util import np_to_torch_bits, run_softmax, torch_bits_to_np

pytestmark = pytest.mark.gpu
FP32, BF16, FP16 = W.FP32, W.BF16, W.FP16


def poison_masked(x, dtype, q_offset, seed):
    """Overwrite every masked entry with NaN / +-inf / large values."""
    rows, cols = x.shape
    xf = W.stored_to_f32(x, dtype).astype(np.float64)
    rng = np.random.default_rng(seed)
    junk = np.array([np.nan, np.inf, -np.inf, 6.0e4, -6.0e4, 0.0])
    j = np.arange(cols)[None, :]
    i = np.arange(rows)[:, None]
    mask = j > i + q_offset
    xf[mask] = junk[rng.integers(0, len(junk), size=int(mask.sum()))]
    return W.to_stored(xf, dtype)


def check_causal(x, dtype, q_offset, scale, y):
    want = fso.softmax_causal_f64(x, dtype, q_offset, scale)
    rep = fso.compare(y, dtype, want)
    assert rep.ok(dtype), (x.shape, dtype, q_offset, scale, rep)
    return rep


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_causal_shape_sweep(dtype):
    shapes = [(1, 1), (5, 8), (33, 24), (64, 64), (100, 1000), (257, 1024), (300, 4096), (70, 16384), (40, 40000),
              (9, 262144), (130, 129), (50, 1001), (20, 100000)]
    for rows, cols in shapes:
        for q_offset in sorted({0, cols - rows, 3, -2, cols, cols // 2}):
            scale = [1.0, 0.5, -1.0, 0.0][(rows + q_offset) % 4]
            x = W.random_case(rows, cols, dtype, seed=rows * 7 + cols, sigma=2.5)
            x = poison_masked(x, dtype, q_offset, seed=cols)
            status, y = run_softmax(x, dtype, scale, causal_q=q_offset)
            assert status == fs.FS_OK, (rows, cols, q_offset, fs.fs_strerror(status), fs.fs_last_cuda_error())
            check_causal(x, dtype, q_offset, scale, y)


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_causal_alignment_inplace_and_special_rows(dtype):
    rows, cols = 40, 2048
    x = W.random_case(rows, cols, dtype, seed=4, sigma=2.0, neg_inf_frac=0.05)
    xf = W.stored_to_f32(x, dtype).astype(np.float64)
    xf[0, 0] = 0.5                      # row 0 keeps this one entry
    xf[3, :4] = [0.0, 1.0, -1.0, 2.0]
    xf[7, 2] = np.nan                   # a kept NaN: whole row NaN, masked part included
    xf[9, 1] = np.inf                   # a kept +inf: same
    xf[11, :12] = -np.inf               # every kept entry masked by the data itself: NaN row
    x = poison_masked(W.to_stored(xf, dtype), dtype, 0, seed=1)
    for kw in ({}, {"offset": 1}, {"offset": 3}, {"inplace": True}):
        status, y = run_softmax(x, dtype, 1.0, causal_q=0, **kw)
        assert status == fs.FS_OK
        check_causal(x, dtype, 0, 1.0, y)
        yf = W.stored_to_f32(y, dtype)
        assert np.all(np.isnan(yf[7])) and np.all(np.isnan(yf[9])) and np.all(np.isnan(yf[11]))
        assert yf[0, 0] == 1.0 and np.all(yf[0, 1:] == 0)
    status, y = run_softmax(x, dtype, 1.0, causal_q=-3)           # rows 0..2 keep nothing
    yf = W.stored_to_f32(y, dtype)
    assert np.all(np.isnan(yf[:3])) and yf[3, 0] == 1.0
    check_causal(x, dtype, -3, 1.0, y)


def test_causal_equals_plain_softmax_on_the_causal_workload():
    """cfg5 carries its mask as -inf in the data: both entry points must agree with the oracle, and
    the causal one must not depend on what the masked entries hold."""
    w = W.WORKLOADS["cfg5"]
    x = W.generate_rows(w, 0, 96)[:, :8192].copy()
    status, a = run_softmax(x, w.dtype, 1.0)
    status, b = run_softmax(x, w.dtype, 1.0, causal_q=0)
    garbage = x.copy()
    garbage[~np.isfinite(garbage)] = np.nan
    status, c = run_softmax(garbage, w.dtype, 1.0, causal_q=0)
    check_causal(x, w.dtype, 0, 1.0, a)
    check_causal(x, w.dtype, 0, 1.0, b)
    assert np.array_equal(b.view(np.uint32), c.view(np.uint32))


def test_causal_full_size_sampled():
    w = W.WORKLOADS["cfg5"]
    free, _ = torch.cuda.mem_get_info()
    if free < 10 * (1 << 30):
        pytest.skip("needs 8 GiB of device memory")
    xd = torch.empty((w.rows, w.cols), dtype=torch.float32, device="cuda")
    step = 2048
    for r0 in range(0, w.rows, step):
        xd[r0:r0 + step].copy_(torch.from_numpy(W.generate_rows(w, r0, r0 + step, threads=8)))
    yd = torch.full_like(xd, float("nan"))
    fs.fs_softmax_causal(xd, yd, w.rows, w.cols, 0, w.dtype, 1.0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    rng = np.random.default_rng(5)
    for i in sorted(set([0, 1, 2, 3, 4, 7, 8, 1023, 1024, 8191, 8192, w.rows - 1] + list(rng.integers(0, w.rows, 50)))):
        x = W.generate_rows(w, i, i + 1)
        want = fso.softmax_f64(x, w.dtype, 1.0)          # the data's own -inf mask equals the causal mask
        rep = fso.compare(yd[i:i + 1].cpu().numpy(), w.dtype, want)
        assert rep.ok(w.dtype), (i, rep)
    assert not bool(torch.isnan(yd).any())
    nz = (yd != 0).sum(dim=1)
    assert bool((nz == torch.arange(1, w.rows + 1, device="cuda")).all())
    assert float((yd.sum(dim=1, dtype=torch.float64) - 1).abs().max()) < 1e-4
