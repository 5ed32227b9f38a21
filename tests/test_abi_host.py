"""Host-side checks that need no GPU: the shared library loads and exports every symbol the header
declares, argument validation answers before any CUDA call, the dispatcher's table, and the loud
failure when no device is usable. No compute happens here."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "fsoftmax.h")


@pytest.fixture(scope="module")
def lib():
    _build.build_library()
    return fs.binding.lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fs_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("fs_softmax", "fs_softmax_ex", "fs_select_kernel", "fs_softmax_host", "fs_copy",
                 "fs_device_status", "fs_release", "fs_last_cuda_error", "fs_strerror", "fs_kernel_name",
                 "fs_version"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    raw = ctypes.CDLL(fs.binding.LIB_PATH)
    for name in declared_functions():
        assert hasattr(raw, name), f"{name} declared in fsoftmax.h but not exported"
    assert "sm_100a" in fs.fs_version()


def test_binding_mirrors_the_header():
    for name in declared_functions():
        assert hasattr(fs, name), f"binding lacks {name}"


def test_enums_match_header():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    for name, value in re.findall(r"(FS_[A-Z0-9_]+)\s*=\s*(\d+)", text):
        assert getattr(fs, name) == int(value), name


def test_constants_match_header():
    text = open(HEADER).read()
    m = re.search(r"#define FS_STATIC_MAX_ROW_BYTES \((\d+) \* (\d+) \* (\d+)\)", text)
    assert m and int(m.group(1)) * int(m.group(2)) * int(m.group(3)) == fs.FS_STATIC_MAX_ROW_BYTES
    m = re.search(r"#define FS_STATIC_SCRATCH_BYTES (\d+)", text)
    assert m and int(m.group(1)) == fs.FS_STATIC_SCRATCH_BYTES
    assert "#define FS_STATIC_MAX_PAIRS ((FS_STATIC_SCRATCH_BYTES - 256) / 8)" in text
    assert fs.FS_STATIC_MAX_PAIRS == (fs.FS_STATIC_SCRATCH_BYTES - 256) // 8


def test_strings(lib):
    assert fs.fs_strerror(fs.FS_OK) == "ok"
    assert "invalid" in fs.fs_strerror(fs.FS_ERR_INVALID_ARG)
    assert [fs.fs_kernel_name(k) for k in range(6)] == ["auto", "warp", "block", "block_tma", "cluster", "generic"]
    assert fs.fs_kernel_name(99) == "unknown"


def test_invalid_arguments_are_rejected_before_any_launch(lib):
    a, b = 0x10000, 0x20000000         # never dereferenced: validation fails first
    bad = fs.FS_ERR_INVALID_ARG
    st = fs.fs_softmax_status
    assert st(a, b, -1, 8, fs.FS_DTYPE_FP32) == bad
    assert st(a, b, 8, -1, fs.FS_DTYPE_FP32) == bad
    assert st(a, b, 8, 8, 3) == bad
    assert st(a, b, 8, 8, -1) == bad
    assert st(0, b, 8, 8, fs.FS_DTYPE_FP32) == bad
    assert st(a, 0, 8, 8, fs.FS_DTYPE_FP32) == bad
    assert st(a, b, 8, 8, fs.FS_DTYPE_FP32, float("nan")) == bad
    assert st(a, b, 8, 8, fs.FS_DTYPE_FP32, float("inf")) == bad
    assert st(a, a + 16, 8, 8, fs.FS_DTYPE_FP32) == bad            # partial overlap
    assert st(a + 16, a, 8, 8, fs.FS_DTYPE_BF16) == bad
    assert st(a, b, 8, 8, fs.FS_DTYPE_FP32, 1.0, None, 6) == bad     # unknown kernel
    assert st(a, b, 8, 8, fs.FS_DTYPE_FP32, 1.0, None, 0, 0, 17) == bad
    assert st(a, b, 1 << 41, 8, fs.FS_DTYPE_FP32) == bad
    # empty problems are fine and launch nothing (null pointers allowed)
    assert st(0, 0, 0, 8, fs.FS_DTYPE_FP32) == fs.FS_OK
    assert st(0, 0, 8, 0, fs.FS_DTYPE_FP16) == fs.FS_OK
    with pytest.raises(fs.FsError):
        fs.fs_softmax(0, b, 8, 8, fs.FS_DTYPE_FP32)
    assert lib.fs_copy(a, b, 24, None) == bad
    assert lib.fs_copy(a + 4, b, 32, None) == bad
    assert lib.fs_copy(0, 0, 0, None) == fs.FS_OK


def test_dispatcher_table(lib):
    k = fs.fs_select_kernel
    F32, BF16, F16 = fs.FS_DTYPE_FP32, fs.FS_DTYPE_BF16, fs.FS_DTYPE_FP16
    # the five benchmark workloads
    assert k(64, 1000, F32) in (fs.FS_KERNEL_WARP, fs.FS_KERNEL_BLOCK)
    assert k(64, 100, F32) == fs.FS_KERNEL_WARP
    assert k(16384, 2048, BF16) in (fs.FS_KERNEL_WARP, fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA)
    assert k(131072, 128, BF16) == fs.FS_KERNEL_WARP
    assert k(256, 262144, BF16) == fs.FS_KERNEL_CLUSTER
    assert k(32768, 32768, F32) in (fs.FS_KERNEL_CLUSTER, fs.FS_KERNEL_BLOCK_TMA)
    # mid-size rows take a block-per-row kernel
    assert k(100, 8192, F32) in (fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA)
    assert k(100, 4096, F16) in (fs.FS_KERNEL_BLOCK, fs.FS_KERNEL_BLOCK_TMA)
    assert k(100, 8192, F16) == fs.FS_KERNEL_CLUSTER        # one block per row, row resident in shared memory
    # ragged rows or misaligned bases take the generic kernel
    assert k(10, 1001, BF16) == fs.FS_KERNEL_GENERIC
    assert k(10, 1023, F32) == fs.FS_KERNEL_GENERIC
    assert k(10, 1024, F32, 4, 16) == fs.FS_KERNEL_GENERIC
    assert k(10, 1024, F32, 16, 8) == fs.FS_KERNEL_GENERIC
    # rows beyond what a 16-block cluster holds in registers fall back too
    assert k(2, 1 << 22, F32) == fs.FS_KERNEL_GENERIC
    assert k(-1, 8, F32) < 0 and k(8, 8, 7) < 0 and k(8, 8, F32, 0, 16) < 0
    # monotone in row size: warp -> block -> cluster -> generic
    order = {fs.FS_KERNEL_WARP: 0, fs.FS_KERNEL_BLOCK: 1, fs.FS_KERNEL_BLOCK_TMA: 1, fs.FS_KERNEL_CLUSTER: 2,
             fs.FS_KERNEL_GENERIC: 3}
    for dt, e in ((F32, 4), (BF16, 2)):
        last = 0
        for log in range(2, 24):
            cur = order[k(4, (1 << log) * 16 // e // 4, dt)]
            assert cur >= last
            last = cur


def test_split_geometry_choice(lib):
    """The split-row geometry: slices of about 32 KiB that are whole chunks (8 vectors per thread), the smallest
    cluster that gets there, any cluster size 1..16 (values fixed by the sweeps the chooser was fitted to)."""
    g = fs.fs_split_geometry
    F32, BF16 = fs.FS_DTYPE_FP32, fs.FS_DTYPE_BF16
    kib = lambda k, e: int(k * 1024) // e
    assert g(kib(32, 2), BF16) == (1, 128, 32768)
    assert g(kib(128, 2), BF16) == (4, 128, 32768)
    assert g(kib(96, 2), BF16) == (3, 128, 32768)                 # not the next power of two with half-empty slices
    assert g(kib(160, 4), F32) == (5, 128, 32768)
    assert g(kib(384, 2), BF16) == (12, 128, 32768)
    assert g(262144, BF16) == (16, 128, 32768)                     # cfg4
    assert g(32768, F32) == (4, 128, 32768)                        # cfg5
    assert g(kib(40, 2), BF16) == (1, 160, 40960)                  # one block, two 20 KiB chunks
    assert g(kib(1024, 2), BF16) == (16, 256, 65536)
    for cols, dt, e in ((kib(24, 2), BF16, 2), (kib(48, 4), F32, 4), (kib(250.5, 2), BF16, 2), (kib(600, 4), F32, 4), (100000, BF16, 2)):
        cs, t, sl = g(cols, dt)
        assert 1 <= cs <= 16 and t % 32 == 0 and 32 <= t <= 256
        assert sl * cs >= cols * e and sl <= 8 * 8 * t * 16          # covers the row; at most 8 chunks of 8 vectors per thread
        assert cs == 16 or sl <= 49152
    assert g(kib(4096, 2), BF16) is None                           # beyond 16 x 192 KiB
    assert g(1001, BF16) is None                                   # not a whole number of vectors
    # every row length the chooser can meet yields a valid geometry
    for nv in list(range(1, 600)) + [1000, 2047, 2048, 2049, 4096, 10000, 65536, 196608]:
        r = g(nv * 8, BF16)
        assert r is not None and r[2] * r[0] >= nv * 16 and r[2] <= 8 * 8 * r[1] * 16, (nv, r)


def test_no_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    x = np.zeros((4, 8), dtype=np.float32)
    # a valid-looking call without a GPU must report a CUDA error, never compute on the host
    assert fs.fs_softmax_status(x.ctypes.data, x.ctypes.data, 4, 8, fs.FS_DTYPE_FP32) == fs.FS_ERR_CUDA
    assert fs.fs_last_cuda_error() != 0
    y = np.full_like(x, 7.0)
    with pytest.raises(fs.FsError):
        fs.fs_softmax_host(x, y, 4, 8, fs.FS_DTYPE_FP32)
    assert np.all(y == 7.0)


def test_missing_library_raises(monkeypatch, tmp_path):
    from paper_2607_24762_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()
