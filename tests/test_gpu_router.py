"""GPU parity of fs_router_topk against the oracle's router step: column indices bit-exact (the
selection is made on the exact inputs on both sides, ties to the lower column), weights within the
fp32 bound of the softmax (|error| <= 1e-6; NaN where the oracle has NaN)."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fso
from paper_2607_24762_b200 import workloads as W

from gpu_util import np_to_torch_bits

pytestmark = pytest.mark.gpu
FP32, BF16, FP16 = W.FP32, W.BF16, W.FP16


def run_router(x, dtype, k, scale, renorm):
    rows, cols = x.shape
    xd = np_to_torch_bits(x).cuda()
    guard = 16
    w = torch.full((rows * k + 2 * guard,), -7.0, dtype=torch.float32, device="cuda")
    idx = torch.full((rows * k + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    st = fs.binding.lib().fs_router_topk(xd.data_ptr(), w.data_ptr() + 4 * guard, idx.data_ptr() + 4 * guard, rows, cols, k,
                                         dtype, scale, int(renorm), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    if st != fs.FS_OK:
        return st, None, None
    wn, inn = w.cpu().numpy(), idx.cpu().numpy()
    assert np.all(wn[:guard] == -7) and np.all(wn[-guard:] == -7) and np.all(inn[:guard] == -7) and np.all(inn[-guard:] == -7)
    return st, wn[guard:-guard].reshape(rows, k), inn[guard:-guard].reshape(rows, k)


def check_router(x, dtype, k, scale, renorm):
    st, w, idx = run_router(x, dtype, k, scale, renorm)
    assert st == fs.FS_OK, fs.fs_strerror(st)
    ww, ii = fso.router_topk_f64(x, dtype, k, scale, renorm)
    nan_rows = np.isnan(ww).any(axis=1)
    assert np.array_equal(np.isnan(w), np.isnan(ww))
    assert np.array_equal(idx, ii), np.argwhere(idx != ii)[:5]
    ok = ~nan_rows
    err = np.abs(w[ok].astype(np.float64) - ww[ok]).max() if ok.any() else 0.0
    assert err <= 1e-6, err
    return err


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_router_sweep(dtype):
    worst = 0.0
    for rows, cols in ((1, 8), (7, 16), (100, 64), (1000, 128), (333, 256), (65, 512), (40, 1024), (50, 24), (9, 40)):
        if (cols * W.ELEM_SIZE[dtype]) % 16:
            continue
        for k in sorted({1, 2, min(8, cols), min(cols, 64)}):
            for scale, renorm in ((1.0, False), (1.0, True), (0.37, True), (-1.0, False), (0.0, True)):
                x = W.random_case(rows, cols, dtype, seed=rows + cols + k, sigma=1.5, neg_inf_frac=0.05)
                worst = max(worst, check_router(x, dtype, k, scale, renorm))
    print(f"router dtype={dtype} max abs weight error {worst:.2e}")


def test_router_ties_and_special_rows():
    cols = 128
    rng = np.random.default_rng(3)
    rows = []
    rows.append(np.round(rng.standard_normal(cols) * 2) / 2)            # heavy ties
    rows.append(np.zeros(cols))                                          # all equal: columns 0..k-1
    r = rng.standard_normal(cols); r[5] = np.nan; rows.append(r)        # NaN row
    r = rng.standard_normal(cols); r[77] = np.inf; rows.append(r)       # +inf wins and poisons
    rows.append(np.full(cols, -np.inf))                                  # nothing finite
    r = np.full(cols, -np.inf); r[100] = 1.0; r[3] = 1.0; rows.append(r)   # two finite, rest masked
    r = rng.standard_normal(cols); r[::2] = -0.0; r[1::2] = 0.0; rows.append(r)   # signed zeros tie
    x = W.to_stored(np.array(rows), BF16)
    for k in (1, 4, 8):
        for renorm in (False, True):
            check_router(x, BF16, k, 1.0, renorm)
            check_router(x, BF16, k, -0.5, renorm)
    _, w, idx = run_router(x, BF16, 4, 1.0, False)
    assert list(idx[1]) == [0, 1, 2, 3] and list(idx[5]) == [3, 100, 0, 1] and list(idx[6]) == [0, 1, 2, 3]


def test_router_both_selection_kernels_agree(monkeypatch):
    """k <= 8 selects with sorting networks in registers; FS_ROUTER_ROUNDS=1 (read per call) keeps the
    kernel that takes one maximum per round. Same columns bit for bit, weights within the parity
    bound of each against the oracle, on tie-heavy and special rows in every dtype."""
    rng = np.random.default_rng(11)
    for dtype in (FP32, BF16, FP16):
        for cols in (8, 16, 64, 128, 256, 1024):
            if (cols * W.ELEM_SIZE[dtype]) % 16:
                continue
            x64 = np.round(rng.standard_normal((37, cols)) * 2) / 2            # heavy ties
            x64[3, :] = 0.0
            x64[5, ::3] = -np.inf
            x64[7, 1] = np.nan
            x = W.to_stored(x64, dtype)
            for k in (1, 3, 8):
                for scale, renorm in ((1.0, True), (-0.7, False), (0.0, True)):
                    monkeypatch.delenv("FS_ROUTER_ROUNDS", raising=False)
                    st_a, w_a, i_a = run_router(x, dtype, k, scale, renorm)
                    check_router(x, dtype, k, scale, renorm)
                    monkeypatch.setenv("FS_ROUTER_ROUNDS", "1")
                    st_b, w_b, i_b = run_router(x, dtype, k, scale, renorm)
                    check_router(x, dtype, k, scale, renorm)
                    assert st_a == st_b == fs.FS_OK and np.array_equal(i_a, i_b)
                    assert np.array_equal(np.isnan(w_a), np.isnan(w_b))
                    assert np.allclose(np.nan_to_num(w_a), np.nan_to_num(w_b), rtol=0, atol=2e-6)
    monkeypatch.delenv("FS_ROUTER_ROUNDS", raising=False)


def test_router_workload_cfg3_top8():
    w = W.WORKLOADS["cfg3"]
    x = W.generate_rows(w, 0, 32768, threads=8)
    check_router(x, w.dtype, 8, 1.0, True)
    check_router(x, w.dtype, 8, 1.0, False)


def test_router_argument_errors():
    L = fs.binding.lib()
    a = torch.zeros(4096, dtype=torch.float32, device="cuda")
    wv = torch.zeros(4096, dtype=torch.float32, device="cuda")
    iv = torch.zeros(4096, dtype=torch.int32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    call = lambda rows, cols, k, dtype=FP32, x=a.data_ptr(): L.fs_router_topk(x, wv.data_ptr(), iv.data_ptr(), rows, cols, k, dtype, 1.0, 0, s)
    assert call(4, 64, 0) == fs.FS_ERR_INVALID_ARG and call(4, 64, 65) == fs.FS_ERR_INVALID_ARG
    assert call(4, 8, 9) == fs.FS_ERR_INVALID_ARG and call(-1, 8, 1) == fs.FS_ERR_INVALID_ARG
    assert call(4, 66, 2) == fs.FS_ERR_UNSUPPORTED                      # row size not a multiple of 16 bytes
    assert call(1, 2048, 2) == fs.FS_ERR_UNSUPPORTED                    # more than 1024 columns
    assert call(4, 64, 2, x=a.data_ptr() + 4) == fs.FS_ERR_UNSUPPORTED
    assert call(0, 64, 2) == fs.FS_OK
    assert L.fs_router_topk(0, wv.data_ptr(), iv.data_ptr(), 4, 64, 2, FP32, 1.0, 0, s) == fs.FS_ERR_INVALID_ARG
    torch.cuda.synchronize()
