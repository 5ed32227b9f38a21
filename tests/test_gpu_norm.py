"""GPU parity of fs_layer_norm and fs_group_norm against the fp64 oracle (oracle/fno.py), element by
element on seeded inputs, through the C ABI. The bar: fp32 |error| <= 2e-6 x the element's error
scale (|gamma| (|x - mu| + mean|x|) / sigma + |beta|: what binary32 statistics can deliver);
bf16/fp16 within one unit of the correctly rounded fp64 value, or within that fp32 bound where
gamma * n and beta cancel."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fno
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


def stored(a64, dtype):
    """float64 values -> stored elements of dtype (one rounding)."""
    from oracle import fso
    return fso.round_from_f64(np.asarray(a64, dtype=np.float64), dtype)


def make_case(rows, cols, dtype, seed, offset=0.0, sigma=1.0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols)) * sigma + offset + rng.standard_normal((rows, 1)) * 0.5
    return stored(x, dtype)


def run_layer(x, dtype, gamma, beta, eps, misalign=0):
    rows, cols = x.shape
    pad = misalign
    xd = np_to_torch_bits(np.concatenate([np.zeros(pad, x.dtype), x.ravel()])).cuda()
    yd = torch.zeros_like(xd)
    gd = None if gamma is None else np_to_torch_bits(gamma).cuda()
    bd = None if beta is None else np_to_torch_bits(beta).cuda()
    esz = W.ELEM_SIZE[dtype]
    fs.fs_layer_norm(xd.data_ptr() + pad * esz, gd, bd, yd.data_ptr() + pad * esz, rows, cols, dtype, eps,
                     torch.cuda.current_stream())
    torch.cuda.synchronize()
    return torch_bits_to_np(yd, dtype)[pad:].reshape(rows, cols)


def check_layer(x, dtype, gamma, beta, eps, **kw):
    from oracle import fso
    y = run_layer(x, dtype, gamma, beta, eps, **kw)
    want = fno.layer_norm_f64(x, dtype, gamma, beta, eps)
    g64 = None if gamma is None else fso.widen(gamma, dtype)[None, :]
    b64 = None if beta is None else fso.widen(beta, dtype)[None, :]
    scale = fno.error_scale(x, dtype, x.shape, g64, b64, eps)
    rep = fno.compare(y, dtype, want, scale)
    assert rep.ok(dtype), (x.shape, dtype, rep)
    return rep


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_layer_norm_shape_sweep(dtype):
    esz = W.ELEM_SIZE[dtype]
    worst = 0.0
    for ci, cols in enumerate([1, 2, 3, 8, 16, 24, 100, 128, 257, 512, 1000, 1024, 1536, 2048, 4096, 5000, 8192, 12288,
                               16384, 40000, 65536, 100000, 262144, 300001]):
        for rows in ((1, 3, 65) if cols <= 16384 else (1, 5)):
            x = make_case(rows, cols, dtype, seed=100 + ci, offset=(ci % 3) * 1.5, sigma=1.0 + (ci % 4))
            affine = ci % 3
            gamma = stored(np.random.default_rng(ci).standard_normal(cols), dtype) if affine >= 1 else None
            beta = stored(np.random.default_rng(ci + 1).standard_normal(cols), dtype) if affine == 1 else None
            rep = check_layer(x, dtype, gamma, beta, 1e-5)
            worst = max(worst, rep.max_rel_err)
    print("layer_norm worst relative error", dtype, worst)


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_layer_norm_row_lengths_across_the_split_geometries(dtype):
    esz = W.ELEM_SIZE[dtype]
    for kb, rows in ((3, 700), (6, 500), (8, 3000), (12, 900), (24, 400), (40, 300), (48, 260), (96, 150), (100, 120), (160, 100),
                     (250.5, 60), (384, 40), (600, 30), (1024, 12), (2048, 5), (3000, 3), (5000, 3), (16384, 2)):
        cols = int(kb * 1024) // esz
        x = make_case(rows, cols, dtype, seed=int(kb), offset=0.25)
        gamma = stored(np.random.default_rng(1).standard_normal(cols) * 0.5 + 1.0, dtype)
        beta = stored(np.random.default_rng(2).standard_normal(cols) * 0.1, dtype)
        check_layer(x, dtype, gamma, beta, 1e-5)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_layer_norm_rows_around_the_four_rows_per_block_kernel(dtype):
    """Rows of 256..704 sixteen-byte vectors take the kernel that works on four rows per block from shared
    memory: both ends of that range and one vector beyond them, row counts that leave a block partly
    empty, with and without gamma and beta."""
    ve = 16 // W.ELEM_SIZE[dtype]
    for k, nvec in enumerate((255, 256, 257, 300, 511, 703, 704, 705)):
        cols = nvec * ve
        for rows in (1, 4, 5, 7, 130):
            x = make_case(rows, cols, dtype, seed=7 * nvec + rows, offset=0.5 * (k % 3), sigma=1.0 + k % 2)
            gamma = stored(np.random.default_rng(nvec).standard_normal(cols) * 0.5 + 1.0, dtype) if k % 2 == 0 or rows == 5 else None
            beta = stored(np.random.default_rng(nvec + 1).standard_normal(cols) * 0.2, dtype) if k % 3 != 1 else None
            check_layer(x, dtype, gamma, beta, 1e-5)


@pytest.mark.parametrize("rows,cols,dtype", [(16384, 1536, BF16), (40000, 2304, BF16), (38000, 4096, FP16), (8192, 4096, FP32)])
def test_layer_norm_at_benchmark_sizes(rows, cols, dtype):
    """The benchmark's layer_norm shapes, and row counts at which the block kernel takes eight rows per
    block (gamma and beta kept in registers, next row requested early). Compared in slabs of rows."""
    from oracle import fso
    rng = np.random.default_rng(rows + cols)
    gamma = stored(rng.standard_normal(cols) * 0.2 + 1.0, dtype)
    beta = stored(rng.standard_normal(cols) * 0.1, dtype)
    x = np.empty((rows, cols), dtype=W.NP_STORE[dtype])
    for r0 in range(0, rows, 4096):
        r1 = min(rows, r0 + 4096)
        x[r0:r1] = stored(rng.standard_normal((r1 - r0, cols)) * 1.5 + 0.25, dtype)
    y = run_layer(x, dtype, gamma, beta, 1e-5)
    g64, b64 = fso.widen(gamma, dtype)[None, :], fso.widen(beta, dtype)[None, :]
    for r0 in range(0, rows, 4096):
        r1 = min(rows, r0 + 4096)
        want = fno.layer_norm_f64(x[r0:r1], dtype, gamma, beta, 1e-5)
        scale = fno.error_scale(x[r0:r1], dtype, (r1 - r0, cols), g64, b64, 1e-5)
        rep = fno.compare(y[r0:r1], dtype, want, scale)
        assert rep.ok(dtype), (r0, rep)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_layer_norm_edge_cases(dtype):
    # constant rows: zero variance, y = beta; eps = 0 with a constant row is 0 * inf = NaN in both
    x = stored(np.full((4, 256), 3.25), dtype)
    beta = stored(np.linspace(-1, 1, 256), dtype)
    gamma = stored(np.linspace(0.5, 2, 256), dtype)
    check_layer(x, dtype, gamma, beta, 1e-5)
    check_layer(x, dtype, None, None, 0.0)
    # large common offset (cancellation in x - mu), tiny variance
    check_layer(make_case(7, 1536, dtype, seed=5, offset=100.0, sigma=0.5), dtype, gamma=None, beta=None, eps=1e-5)
    # NaN / inf poison their row only
    x = make_case(5, 4096, dtype, seed=6)
    xf = x.copy()
    nan_bits = np.float32(np.nan) if dtype == FP32 else np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    inf_bits = np.float32(np.inf) if dtype == FP32 else np.uint16(0x7F80 if dtype == BF16 else 0x7C00)
    xf[1, 17] = nan_bits
    xf[3, 4000] = inf_bits
    check_layer(xf, dtype, None, None, 1e-5)
    # misaligned base and ragged columns take the generic kernel
    check_layer(make_case(9, 1001, dtype, seed=8), dtype, stored(np.ones(1001) * 1.5, dtype), None, 1e-5)
    check_layer(make_case(9, 1024, dtype, seed=9), dtype, None, None, 1e-5, misalign=1)
    # in place
    x = make_case(33, 2048, dtype, seed=10)
    xd = np_to_torch_bits(x.copy()).cuda()
    fs.fs_layer_norm(xd, None, None, xd, 33, 2048, dtype, 1e-5, torch.cuda.current_stream())
    torch.cuda.synchronize()
    y = torch_bits_to_np(xd, dtype).reshape(33, 2048)
    rep = fno.compare(y, dtype, fno.layer_norm_f64(x, dtype), fno.error_scale(x, dtype, x.shape))
    assert rep.ok(dtype)
    # empty problems
    fs.fs_layer_norm(None, None, None, None, 0, 128, dtype)
    fs.fs_layer_norm(None, None, None, None, 128, 0, dtype)


def test_layer_norm_rejects_bad_arguments():
    a, b = 0x10000, 0x2000000
    L = fs.binding.lib()
    bad = fs.FS_ERR_INVALID_ARG
    assert L.fs_layer_norm(a, None, None, b, -1, 8, FP32, 1e-5, None) == bad
    assert L.fs_layer_norm(a, None, None, b, 8, 8, 7, 1e-5, None) == bad
    assert L.fs_layer_norm(a, None, None, b, 8, 8, FP32, -1.0, None) == bad
    assert L.fs_layer_norm(a, None, None, b, 8, 8, FP32, float("nan"), None) == bad
    assert L.fs_layer_norm(None, None, None, b, 8, 8, FP32, 1e-5, None) == bad
    assert L.fs_layer_norm(a, None, None, a + 16, 8, 8, FP32, 1e-5, None) == bad
    assert L.fs_group_norm(a, None, None, b, 2, 6, 4, 4, FP32, 1e-5, None) == bad      # groups does not divide channels
    assert L.fs_group_norm(a, None, None, b, 2, 6, 4, 0, FP32, 1e-5, None) == bad


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_group_norm(dtype):
    from oracle import fso
    for ci, (n, ch, sp, groups) in enumerate([(2, 8, 16, 4), (1, 32, 64, 32), (3, 64, 256, 32), (2, 128, 1024, 32), (1, 512, 4096, 32),
                                              (1, 256, 16384, 32), (2, 6, 5, 3), (1, 12, 1000, 4), (1, 4, 100000, 2),
                                              (1, 128, 65536, 32), (1, 32, 8, 1),
                                              (1, 4, 900000, 2), (2, 2, 1 << 21, 1)]):      # rows beyond a cluster's shared memory: two-kernel path
        rng = np.random.default_rng(40 + ci)
        x64 = rng.standard_normal((n, ch, sp)) * (1 + rng.random((1, ch, 1)) * 2) + rng.standard_normal((1, ch, 1))
        x = stored(x64, dtype)
        for affine in (True, False):
            gamma = stored(rng.standard_normal(ch) * 0.5 + 1, dtype) if affine else None
            beta = stored(rng.standard_normal(ch) * 0.2, dtype) if affine else None
            xd = np_to_torch_bits(x).cuda()
            yd = torch.zeros_like(xd)
            fs.fs_group_norm(xd, None if gamma is None else np_to_torch_bits(gamma).cuda(),
                             None if beta is None else np_to_torch_bits(beta).cuda(), yd, n, ch, sp, groups, dtype, 1e-5,
                             torch.cuda.current_stream())
            torch.cuda.synchronize()
            y = torch_bits_to_np(yd, dtype).reshape(n, ch, sp)
            want = fno.group_norm_f64(x, dtype, groups, gamma, beta, 1e-5)
            cpg = ch // groups
            gfull = None if gamma is None else np.repeat(fso.widen(gamma, dtype), sp).reshape(1, ch * sp).repeat(n, 0).reshape(n * groups, cpg * sp)
            bfull = None if beta is None else np.repeat(fso.widen(beta, dtype), sp).reshape(1, ch * sp).repeat(n, 0).reshape(n * groups, cpg * sp)
            scale = fno.error_scale(x, dtype, (n * groups, cpg * sp), gfull, bfull, 1e-5)
            rep = fno.compare(y, dtype, want, scale.reshape(n, ch, sp))
            assert rep.ok(dtype), ((n, ch, sp, groups), affine, rep)
