"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle, element by
element on the same seeded inputs. The bar is the one the benchmark contract states: fp32
max |delta| <= 1e-6 against the unrounded fp64 value; bf16/fp16 within 1 ulp of the fp64 value
rounded once to the format; exact +0 where the oracle has exact 0; NaN where it has NaN."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fso
from paper_2607_24762_b200 import workloads as W

from gpu_util import check, np_to_torch_bits, run_softmax, torch_bits_to_np

pytestmark = pytest.mark.gpu

FP32, BF16, FP16 = W.FP32, W.BF16, W.FP16
ALL_KERNELS = [fs.FS_KERNEL_WARP, fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA, fs.FS_KERNEL_CLUSTER,
               fs.FS_KERNEL_GENERIC]
SCALES = [1.0, 0.5, 128 ** -0.5, -1.0, 0.0]


@pytest.fixture(scope="module", autouse=True)
def built_library():
    from paper_2607_24762_b200 import _build
    _build.build_library()
    assert "libfsoftmax" in fs.binding.LIB_PATH      # the normal build, or the checked one (FSOFTMAX_LIB)
    yield
    assert fs.fs_device_status() == fs.FS_OK       # no bounded wait expired in any test


def sweep_case(rows, cols, dtype, kernel, scale, seed, **kw):
    x = W.random_case(rows, cols, dtype, seed=seed, sigma=2.5, neg_inf_frac=0.03 if scale > 0 else 0.0)
    status, y = run_softmax(x, dtype, scale, kernel, **kw)
    if status == fs.FS_ERR_UNSUPPORTED and kernel != fs.FS_KERNEL_AUTO:
        return None
    assert status == fs.FS_OK, (fs.fs_strerror(status), fs.fs_last_cuda_error())
    return check(x, dtype, scale, y)


# ---------------------------------------------------------------------------------------------
# shape sweep: every kernel forced on every shape it accepts; auto on everything
# ---------------------------------------------------------------------------------------------

COLS_SMALL = [1, 2, 3, 4, 7, 8, 15, 16, 17, 31, 32, 33, 127, 128, 129, 1000, 1023, 1024, 1025, 2048, 4095, 4096, 4097]
COLS_LARGE = [8192, 32768, 65536, 100000, 262144, 262145]


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
@pytest.mark.parametrize("kernel", [fs.FS_KERNEL_AUTO] + ALL_KERNELS)
def test_shape_sweep_small(dtype, kernel):
    ran = 0
    for ci, cols in enumerate(COLS_SMALL):
        for rows in (1, 2, 3, 63, 64, 65, 1000) if ci % 3 == 0 else (1, 65, 257):
            scale = SCALES[(ci + rows) % len(SCALES)]
            rep = sweep_case(rows, cols, dtype, kernel, scale, seed=1000 + ci)
            ran += rep is not None
    assert ran > 0 or kernel == fs.FS_KERNEL_CLUSTER


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
@pytest.mark.parametrize("kernel", [fs.FS_KERNEL_AUTO] + ALL_KERNELS)
def test_shape_sweep_large(dtype, kernel):
    ran = 0
    for ci, cols in enumerate(COLS_LARGE):
        for rows in (1, 5, 37):
            scale = SCALES[(ci + rows) % 3]
            rep = sweep_case(rows, cols, dtype, kernel, scale, seed=2000 + ci)
            ran += rep is not None
    assert ran > 0 or kernel == fs.FS_KERNEL_WARP          # rows this long exceed a warp's registers


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_very_long_rows(dtype):
    for cols, rows in ((1 << 20, 3), ((1 << 21) + 8, 2)):
        assert sweep_case(rows, cols, dtype, fs.FS_KERNEL_AUTO, 1.0, seed=31) is not None


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_rows_beyond_a_cluster_take_the_two_kernel_path(dtype):
    """Rows of 4-16 MiB (no cluster's shared memory holds them): segments over two kernels, partial pairs through a
    stream-ordered scratch buffer. Positive, negative and zero scale, -inf entries, a NaN row, in place."""
    cols = (1 << 21) + 24 if dtype != FP32 else (1 << 20) + 12
    for rows, scale in ((3, 1.0), (2, -0.5), (1, 0.0)):
        x = W.random_case(rows, cols, dtype, seed=90 + rows, sigma=3.0, neg_inf_frac=0.02 if scale > 0 else 0.0)
        status, y = run_softmax(x, dtype, scale)
        assert status == fs.FS_OK
        check(x, dtype, scale, y)
    x = W.random_case(2, cols, dtype, seed=99, sigma=2.0)
    x[1, 12345] = np.float32(np.nan) if dtype == FP32 else np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)
    status, y = run_softmax(x, dtype, 1.0, inplace=True)
    assert status == fs.FS_OK
    check(x, dtype, 1.0, y)


@pytest.mark.parametrize("kernel,threads,cluster", [
    (fs.FS_KERNEL_BLOCK, 32, 0), (fs.FS_KERNEL_BLOCK, 64, 0), (fs.FS_KERNEL_BLOCK, 128, 0), (fs.FS_KERNEL_BLOCK, 512, 0),
    (fs.FS_KERNEL_BLOCK, 1024, 0), (fs.FS_KERNEL_BLOCK_TMA, 32, 0), (fs.FS_KERNEL_BLOCK_TMA, 96, 0),
    (fs.FS_KERNEL_BLOCK_TMA, 256, 0), (fs.FS_KERNEL_BLOCK_TMA, 1024, 0),
    (fs.FS_KERNEL_CLUSTER, 0, 1), (fs.FS_KERNEL_CLUSTER, 0, 2), (fs.FS_KERNEL_CLUSTER, 0, 4), (fs.FS_KERNEL_CLUSTER, 0, 8),
    (fs.FS_KERNEL_CLUSTER, 0, 16), (fs.FS_KERNEL_CLUSTER, 128, 4), (fs.FS_KERNEL_CLUSTER, 256, 2),
    (fs.FS_KERNEL_CLUSTER, 32, 8), (fs.FS_KERNEL_CLUSTER, 0, 3), (fs.FS_KERNEL_CLUSTER, 96, 5), (fs.FS_KERNEL_CLUSTER, 160, 6),
    (fs.FS_KERNEL_CLUSTER, 0, 7), (fs.FS_KERNEL_CLUSTER, 192, 9), (fs.FS_KERNEL_CLUSTER, 0, 11), (fs.FS_KERNEL_CLUSTER, 224, 12),
    (fs.FS_KERNEL_CLUSTER, 0, 13), (fs.FS_KERNEL_CLUSTER, 64, 15), (fs.FS_KERNEL_WARP, 128, 0), (fs.FS_KERNEL_WARP, 32, 0),
    (fs.FS_KERNEL_GENERIC, 32, 0), (fs.FS_KERNEL_GENERIC, 1024, 0),
])
def test_every_launch_geometry_the_dispatcher_can_pick(kernel, threads, cluster):
    ran = 0
    for dtype in (FP32, BF16, FP16):
        for cols in (8, 24, 520, 2048, 5000 * 8, 16384, 65536):
            for rows in (1, 33, 300):
                if rows * cols > 4_000_000:
                    continue
                rep = sweep_case(rows, cols, dtype, kernel, 0.7, seed=77, threads=threads, cluster=cluster)
                ran += rep is not None
    assert ran > 0


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_split_row_geometry_choice_over_row_lengths(dtype):
    """Row lengths from 8 KiB to 1.5 MiB, multiples of 32 KiB and not: the dispatcher's choice of cluster size
    (any of 1..16) and block size (96..256 threads) for each, with more rows than resident clusters so
    that the L2 prefetch of later rows runs."""
    esz = 4 if dtype == FP32 else 2
    for kb, rows in ((8, 3000), (12, 2500), (20, 1500), (24, 1200), (40, 900), (48, 800), (62.5, 600), (80, 500), (96, 400),
                     (100, 400), (160, 260), (192, 230), (250.5, 150), (296.75, 130), (384, 100), (600, 70), (768, 60), (1536, 30)):
        cols = int(kb * 1024) // esz
        rep = sweep_case(rows, cols, dtype, fs.FS_KERNEL_AUTO, 1.0, seed=int(kb * 4))
        assert rep is not None


# ---------------------------------------------------------------------------------------------
# alignment, aliasing, determinism
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_misaligned_bases_and_odd_columns(dtype):
    for offset in (1, 2, 3, 5):
        for cols in (8, 1000, 1024, 4099):
            x = W.random_case(9, cols, dtype, seed=offset * 100 + cols, sigma=2.0)
            status, y = run_softmax(x, dtype, 1.0, offset=offset)
            assert status == fs.FS_OK
            check(x, dtype, 1.0, y)
    x = W.random_case(4, 1024, dtype, seed=5)
    status, _ = run_softmax(x, dtype, 1.0, fs.FS_KERNEL_WARP, offset=1)
    assert status == fs.FS_ERR_UNSUPPORTED                    # fast kernels refuse a misaligned base
    status, _ = run_softmax(W.random_case(4, 1023, dtype, seed=5), dtype, 1.0, fs.FS_KERNEL_BLOCK_TMA)
    assert status == fs.FS_ERR_UNSUPPORTED


@pytest.mark.parametrize("kernel", [fs.FS_KERNEL_AUTO] + ALL_KERNELS)
def test_in_place(kernel):
    for dtype, rows, cols in ((FP32, 70, 1000), (BF16, 33, 2048), (FP16, 300, 128), (BF16, 5, 65536), (FP32, 3, 40000)):
        x = W.random_case(rows, cols, dtype, seed=9, sigma=2.0)
        status, y = run_softmax(x, dtype, 1.0, kernel, inplace=True)
        if status == fs.FS_ERR_UNSUPPORTED:
            continue
        assert status == fs.FS_OK
        check(x, dtype, 1.0, y)


def test_two_runs_are_bit_identical():
    for name in ("cfg1",):
        w = W.WORKLOADS[name]
        x = W.generate(w)
        _, a = run_softmax(x, w.dtype, w.scale_f32)
        _, b = run_softmax(x, w.dtype, w.scale_f32)
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))
    for kernel, rows, cols, dtype in ((fs.FS_KERNEL_CLUSTER, 40, 65536, BF16), (fs.FS_KERNEL_BLOCK_TMA, 500, 4096, FP16),
                                      (fs.FS_KERNEL_WARP, 5000, 128, BF16), (fs.FS_KERNEL_GENERIC, 50, 3001, FP32)):
        x = W.random_case(rows, cols, dtype, seed=3, sigma=3.0)
        _, a = run_softmax(x, dtype, 1.0, kernel)
        _, b = run_softmax(x, dtype, 1.0, kernel)
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


def test_runs_on_a_side_stream():
    s = torch.cuda.Stream()
    x = W.random_case(128, 2048, BF16, seed=1)
    with torch.cuda.stream(s):
        status, y = run_softmax(x, BF16, 1.0, stream=s)
    assert status == fs.FS_OK
    check(x, BF16, 1.0, y)


# ---------------------------------------------------------------------------------------------
# special values
# ---------------------------------------------------------------------------------------------

def special_rows(cols, dtype):
    big = {FP32: 3.0e38, BF16: 3.0e38, FP16: 65504.0}[dtype]
    rng = np.random.default_rng(cols)
    base = rng.standard_normal(cols) * 2.0
    rows = []
    r = base.copy(); r[cols // 2:] = -np.inf; rows.append(r)                      # trailing mask (causal)
    r = base.copy(); r[:cols // 2] = -np.inf; rows.append(r)                      # leading mask
    r = np.full(cols, -np.inf); r[cols - 1] = 0.25; rows.append(r)                # a single finite entry
    rows.append(np.full(cols, -np.inf))                                           # fully masked -> NaN
    r = base.copy(); r[cols // 3] = np.inf; rows.append(r)                        # +inf -> NaN
    r = base.copy(); r[0] = np.nan; rows.append(r)                                # NaN first
    r = base.copy(); r[cols - 1] = np.nan; rows.append(r)                         # NaN last
    r = base.copy(); r[cols // 2] = 1000.0 if dtype != FP16 else 60000.0; rows.append(r)   # dominant entry
    rows.append(np.full(cols, big))                                               # huge and equal
    r = np.full(cols, -big); r[cols // 4] = big; rows.append(r)                   # full dynamic range
    rows.append(np.zeros(cols))                                                   # uniform
    rows.append(np.linspace(-110.0, 0.0, cols))                                   # reaches fp32's subnormal outputs
    rows.append(base)
    return W.to_stored(np.array(rows), dtype)


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
@pytest.mark.parametrize("kernel", [fs.FS_KERNEL_AUTO] + ALL_KERNELS)
def test_special_values(dtype, kernel):
    ran = 0
    for cols in (8, 64, 1000, 4096, 16384, 131072):
        x = special_rows(cols, dtype)
        for scale in (1.0, 0.125):
            status, y = run_softmax(x, dtype, scale, kernel)
            if status == fs.FS_ERR_UNSUPPORTED and kernel != fs.FS_KERNEL_AUTO:
                continue
            assert status == fs.FS_OK
            rep = check(x, dtype, scale, y)
            ran += 1
            yf = W.stored_to_f32(y, dtype)
            assert np.all(np.isnan(yf[3])) and np.all(np.isnan(yf[4])) and np.all(np.isnan(yf[5])) and np.all(np.isnan(yf[6]))
            assert np.all(yf[0, cols // 2:] == 0) and yf[2, cols - 1] == 1.0
            assert rep.nan_mismatch == 0 and rep.zero_mismatch == 0
    assert ran > 0


@pytest.mark.parametrize("dtype", [FP32, BF16, FP16])
def test_negative_and_zero_scale(dtype):
    for cols in (8, 128, 2048, 8192, 65536):
        x = W.random_case(6, cols, dtype, seed=cols, sigma=3.0)
        for scale in (-1.0, -0.37, 0.0):
            for kernel in [fs.FS_KERNEL_AUTO] + ALL_KERNELS:
                status, y = run_softmax(x, dtype, scale, kernel)
                if status == fs.FS_ERR_UNSUPPORTED:
                    continue
                check(x, dtype, scale, y)
        # with a negative scale a -inf entry becomes +inf and poisons its row; +inf becomes a mask
        xs = W.stored_to_f32(x, dtype).astype(np.float64)
        xs[1, 0] = -np.inf
        xs[2, cols - 1] = np.inf
        xs = W.to_stored(xs, dtype)
        status, y = run_softmax(xs, dtype, -1.0)
        rep = check(xs, dtype, -1.0, y)
        yf = W.stored_to_f32(y, dtype)
        assert np.all(np.isnan(yf[1])) and yf[2, cols - 1] == 0 and not np.isnan(yf[2]).any() and rep.nan_mismatch == 0
        status, y = run_softmax(xs, dtype, 0.0)                  # 0 * inf = NaN
        check(xs, dtype, 0.0, y)


@pytest.mark.parametrize("dtype", [BF16, FP16])
def test_rows_around_the_four_rows_per_block_kernel(dtype):
    """16-bit rows above 4 KiB up to 14 KiB (257..896 sixteen-byte vectors, except 384 and 512) take the kernel that
    works on four rows per block from shared memory, a warp per row: both ends of the range and its two holes, one
    vector to either side, row counts that leave a block partly empty, both signs of the scale and zero, in place,
    special values."""
    for ci, nvec in enumerate((256, 257, 300, 383, 384, 385, 511, 512, 513, 700, 895, 896, 897)):
        cols = nvec * 8
        chosen = fs.fs_select_kernel(5, cols, dtype)
        in_range = 256 < nvec <= 896 and nvec not in (384, 512)
        assert (chosen == fs.FS_KERNEL_BLOCK_TMA) == in_range, (nvec, chosen)
        for rows, scale in ((1, 1.0), (5, 0.125), (7, -0.5), (64, 1.0), (3, 0.0)):
            x = W.random_case(rows, cols, dtype, seed=400 + ci + rows, sigma=3.0, neg_inf_frac=0.02 if scale > 0 else 0.0)
            status, y = run_softmax(x, dtype, scale, inplace=(ci + rows) % 3 == 0)
            assert status == fs.FS_OK
            check(x, dtype, scale, y)
    cols = 700 * 8
    x = W.random_case(6, cols, dtype, seed=77, sigma=2.0)
    ninf = np.uint16(0xFF80 if dtype == BF16 else 0xFC00)
    x[1, :] = ninf                                                   # only masked entries: NaN row
    x[2, 1234] = np.uint16(0x7FC0 if dtype == BF16 else 0x7E00)     # NaN
    x[3, 4321] = np.uint16(0x7F80 if dtype == BF16 else 0x7C00)     # +inf
    x[4, 1:] = ninf                                                  # one finite entry: exactly [1, 0, 0, ...]
    status, y = run_softmax(x, dtype, 1.0)
    rep = check(x, dtype, 1.0, y)
    yf = W.stored_to_f32(y, dtype)
    assert np.all(np.isnan(yf[1:4])) and yf[4, 0] == 1.0 and np.all(y[4, 1:] == 0) and rep.nan_mismatch == 0
    if dtype == BF16:                                                # results below 2^-126 are kept
        row = np.linspace(-91.0, -87.0, cols)
        row[0] = 0.0
        xs = W.to_stored(np.array([row, row[::-1].copy(), row]), BF16)
        status, y = run_softmax(xs, BF16, 1.0)
        check(xs, BF16, 1.0, y)
        assert np.count_nonzero((y[0] > 0) & (y[0] < 0x0080)) > 50


def test_bf16_subnormal_outputs_are_not_flushed():
    """Outputs below 2^-126 are representable bf16 subnormals; the 1-ulp rule applies there too."""
    cols = 256
    row = np.linspace(-91.0, -87.0, cols)
    row[0] = 0.0
    x = W.to_stored(np.array([row, row[::-1].copy()]), BF16)
    for kernel in [fs.FS_KERNEL_AUTO] + ALL_KERNELS:
        status, y = run_softmax(x, BF16, 1.0, kernel)
        if status == fs.FS_ERR_UNSUPPORTED:
            continue
        check(x, BF16, 1.0, y)
        assert np.count_nonzero((y[0] > 0) & (y[0] < 0x0080)) > 50      # subnormal bit patterns present


# ---------------------------------------------------------------------------------------------
# the five workloads, in the launch configuration the dispatcher (and so the benchmark) uses
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
def test_workload_full_parity(name):
    w = W.WORKLOADS[name]
    x = W.generate(w, threads=8)
    xd = np_to_torch_bits(x).cuda()
    yd = torch.empty_like(xd)
    fs.fs_softmax(xd, yd, w.rows, w.cols, w.dtype, w.scale_f32, torch.cuda.current_stream())
    torch.cuda.synchronize()
    y = torch_bits_to_np(yd, w.dtype)
    worst_abs, worst_ulp = 0.0, 0
    step = max(1, (1 << 22) // w.cols)
    for r0 in range(0, w.rows, step):
        rep = check(x[r0:r0 + step], w.dtype, w.scale_f32, y[r0:r0 + step])
        worst_abs, worst_ulp = max(worst_abs, rep.max_abs_err), max(worst_ulp, rep.max_ulp)
    print(f"{name}: kernel={fs.fs_kernel_name(fs.fs_select_kernel(w.rows, w.cols, w.dtype))} "
          f"max_abs={worst_abs:.3e} max_ulp={worst_ulp}")
    if name == "cfg4":
        xf = W.stored_to_f32(x[:8], w.dtype)
        assert np.all(y[:8][xf == W.SPIKE_VALUE] == 0x3E00)        # bf16(0.125) on every spike


def test_workload_cfg5_full_size_every_element():
    """All 2^30 elements of the causal workload against the oracle, for fs_softmax on the masked data and for
    fs_softmax_causal(q_offset=0) on the same data with the masked entries replaced by 1e30 (which it must never
    look at): the oracle runs over every row, on all host cores, in pieces of 128 rows."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    w = W.WORKLOADS["cfg5"]
    free, _ = torch.cuda.mem_get_info()
    if free < 10 * (1 << 30):
        pytest.skip("needs 8 GiB of device memory")
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    x = np.empty((w.rows, w.cols), dtype=np.float32)
    xd = torch.empty((w.rows, w.cols), dtype=torch.float32, device="cuda")
    slab = 2048
    for r0 in range(0, w.rows, slab):                             # generate and upload in slabs
        x[r0:r0 + slab] = W.generate_rows(w, r0, r0 + slab, threads=min(8, cores))
        xd[r0:r0 + slab].copy_(torch.from_numpy(x[r0:r0 + slab]))
    yd = torch.empty_like(xd)
    fs.fs_softmax(xd, yd, w.rows, w.cols, w.dtype, w.scale_f32, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    y_plain = yd.cpu().numpy()
    for r0 in range(0, w.rows, slab):
        xd[r0:r0 + slab].nan_to_num_(neginf=1e30)                 # what the causal entry point must not read
    yd.fill_(float("nan"))
    fs.fs_softmax_causal(xd, yd, w.rows, w.cols, 0, w.dtype, w.scale_f32, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    y_causal = yd.cpu().numpy()
    del xd, yd
    piece = 128

    def work(r0):
        want = fso.softmax_f64(x[r0:r0 + piece], w.dtype, w.scale_f32)
        return (fso.compare(y_plain[r0:r0 + piece], w.dtype, want), fso.compare(y_causal[r0:r0 + piece], w.dtype, want))

    with ThreadPoolExecutor(max_workers=cores) as ex:
        reps = list(ex.map(work, range(0, w.rows, piece)))
    for name, k in (("fs_softmax", 0), ("fs_softmax_causal", 1)):
        rs = [r[k] for r in reps]
        n = sum(r.n_compared for r in rs)
        worst = max(r.max_abs_err for r in rs)
        print(f"cfg5 {name}: kernel={fs.fs_kernel_name(fs.fs_select_kernel(w.rows, w.cols, w.dtype))} "
              f"n_compared={n} (2^30 = {1 << 30}) max_abs={worst:.3e} on {cores} host threads")
        assert n == w.rows * w.cols
        assert all(r.ok(w.dtype) for r in rs), [r for r in rs if not r.ok(w.dtype)][:3]
    assert y_plain[0, 0] == 1.0 and y_causal[0, 0] == 1.0


# ---------------------------------------------------------------------------------------------
# host entry point, copy kernel
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,rows,cols", [(FP32, 64, 1000), (BF16, 20000, 2048), (FP16, 3, 9), (BF16, 2, 262144),
                                             (FP32, 100, 100000)])
def test_host_entry_point(dtype, rows, cols):
    x = W.random_case(rows, cols, dtype, seed=rows, sigma=2.0, neg_inf_frac=0.01)
    y = np.empty_like(x)
    fs.fs_softmax_host(x, y, rows, cols, dtype, 0.5)
    step = max(1, (1 << 22) // cols)
    for r0 in range(0, rows, step):
        check(x[r0:r0 + step], dtype, 0.5, y[r0:r0 + step])
    # pinned memory, same result
    xp = torch.from_numpy(x.view(np.int16) if dtype != FP32 else x).pin_memory()
    yp = torch.empty_like(xp).pin_memory()
    fs.fs_softmax_host(xp, yp, rows, cols, dtype, 0.5)
    assert np.array_equal(yp.numpy().view(np.uint8), y.view(np.uint8))
    fs.fs_release()


def test_copy_kernel_is_exact():
    for n in (16, 4096, (1 << 24) + 16 * 13):
        a = torch.randint(0, 255, (n,), dtype=torch.uint8, device="cuda")
        b = torch.zeros_like(a)
        fs.fs_copy(a, b, n, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert torch.equal(a, b)


def test_dispatcher_choice_runs_for_each_workload_shape():
    for w in W.WORKLOADS.values():
        k = fs.fs_select_kernel(w.rows, w.cols, w.dtype)
        assert k in (fs.FS_KERNEL_WARP, fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA, fs.FS_KERNEL_CLUSTER)
        x = W.generate_rows(w, 0, min(w.rows, 8))
        status, y = run_softmax(x, w.dtype, w.scale_f32, k)
        assert status == fs.FS_OK
        check(x, w.dtype, w.scale_f32, y)
