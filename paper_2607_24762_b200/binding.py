"""Thin ctypes binding of libfsoftmax's C ABI (see include/fsoftmax.h).

Argument marshalling only: every step of the softmax runs in the CUDA library. Functions carry
the C entry points' names. Device buffers may be given as torch CUDA tensors (their ``data_ptr``
is passed) or as raw integer addresses; host buffers as numpy arrays or torch CPU tensors.
There is no fallback: if the shared library is missing, or no CUDA device is usable, calls raise.
"""
from __future__ import annotations

import ctypes
import os
import threading

FS_DTYPE_FP32, FS_DTYPE_BF16, FS_DTYPE_FP16 = 0, 1, 2
FS_OK, FS_ERR_INVALID_ARG, FS_ERR_UNSUPPORTED, FS_ERR_CUDA, FS_ERR_DEVICE_TIMEOUT, FS_ERR_DEVICE_BOUNDS = 0, 1, 2, 3, 4, 5
FS_KERNEL_AUTO, FS_KERNEL_WARP, FS_KERNEL_BLOCK, FS_KERNEL_BLOCK_TMA, FS_KERNEL_CLUSTER, FS_KERNEL_GENERIC = range(6)
FS_STATIC_MAX_ROW_BYTES = 16 * 192 * 1024
FS_STATIC_SCRATCH_BYTES = 65536
FS_STATIC_MAX_PAIRS = (FS_STATIC_SCRATCH_BYTES - 256) // 8
FS_ROUTER_MAX_K = 64
KERNELS = {"auto": 0, "warp": 1, "block": 2, "block_tma": 3, "cluster": 4, "generic": 5}

_HERE = os.path.dirname(os.path.abspath(__file__))
# FSOFTMAX_LIB (read at import) selects another build of the same library, e.g. the checked one
# (libfsoftmax_debug.so, see _build.build_library(debug=True)); there is still no fallback.
LIB_PATH = os.environ.get("FSOFTMAX_LIB") or os.path.join(_HERE, "libfsoftmax.so")
_lock = threading.Lock()
_lib = None


class FsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().fs_strerror(status).decode()
        if status == FS_ERR_CUDA:
            msg += f" [cudaError {lib().fs_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} (status {status})")


def lib() -> ctypes.CDLL:
    """Load libfsoftmax.so (built in-tree by ``_build.build_library``). Raises if it is missing."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                raise RuntimeError(
                    f"{LIB_PATH} is missing: build it with "
                    "`python -c 'import __graft_entry__ as g; g.build()'` (needs nvcc). "
                    "There is no CPU or PyTorch fallback.")
            L = ctypes.CDLL(LIB_PATH)
            vp, i64, ci, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
            L.fs_softmax.argtypes = [vp, vp, i64, i64, ci, f32, vp]
            L.fs_softmax.restype = ci
            L.fs_softmax_ex.argtypes = [vp, vp, i64, i64, ci, f32, vp, ci, ci, ci]
            L.fs_softmax_ex.restype = ci
            L.fs_softmax_causal.argtypes = [vp, vp, i64, i64, i64, ci, f32, vp]
            L.fs_softmax_causal.restype = ci
            L.fs_router_topk.argtypes = [vp, vp, vp, i64, i64, ci, ci, f32, ci, vp]
            L.fs_router_topk.restype = ci
            L.fs_log_softmax.argtypes = [vp, vp, i64, i64, ci, f32, vp]
            L.fs_log_softmax.restype = ci
            L.fs_softmax_f32out.argtypes = [vp, vp, i64, i64, ci, f32, vp]
            L.fs_softmax_f32out.restype = ci
            L.fs_softmax_masked.argtypes = [vp, vp, vp, i64, i64, i64, i64, ci, f32, vp]
            L.fs_softmax_masked.restype = ci
            L.fs_softmax_backward.argtypes = [vp, vp, vp, i64, i64, ci, f32, vp]
            L.fs_softmax_backward.restype = ci
            L.fs_layer_norm.argtypes = [vp, vp, vp, vp, i64, i64, ci, f32, vp]
            L.fs_layer_norm.restype = ci
            L.fs_group_norm.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, ci, f32, vp]
            L.fs_group_norm.restype = ci
            L.fs_split_geometry.argtypes = [i64, ci, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(i64)]
            L.fs_split_geometry.restype = ci
            L.fs_select_kernel.argtypes = [i64, i64, ci, ci, ci]
            L.fs_select_kernel.restype = ci
            L.fs_softmax_host.argtypes = [vp, vp, i64, i64, ci, f32]
            L.fs_softmax_host.restype = ci
            L.fs_softmax_static.argtypes = [vp, vp, i64, i64, ci, f32, vp]
            L.fs_softmax_static.restype = ci
            L.fs_static_status.argtypes = []
            L.fs_static_status.restype = ci
            L.fs_debug_set_wait_polls.argtypes = [ci]
            L.fs_debug_set_wait_polls.restype = ci
            L.fs_debug_wait_probe.argtypes = [vp]
            L.fs_debug_wait_probe.restype = ci
            L.fs_debug_softmax_expire.argtypes = [vp, vp, i64, i64, ci, f32, vp, ci, ci]
            L.fs_debug_softmax_expire.restype = ci
            L.fs_debug_checked_build.argtypes = []
            L.fs_debug_checked_build.restype = ci
            L.fs_debug_bad_address.argtypes = [ctypes.POINTER(ctypes.c_uint64)]
            L.fs_debug_bad_address.restype = ci
            L.fs_debug_shrink_writable.argtypes = [i64]
            L.fs_debug_shrink_writable.restype = ci
            L.fs_copy.argtypes = [vp, vp, i64, vp]
            L.fs_copy.restype = ci
            L.fs_device_status.argtypes = []
            L.fs_device_status.restype = ci
            L.fs_release.argtypes = []
            L.fs_release.restype = ci
            L.fs_last_cuda_error.argtypes = []
            L.fs_last_cuda_error.restype = ci
            L.fs_strerror.argtypes = [ci]
            L.fs_strerror.restype = ctypes.c_char_p
            L.fs_kernel_name.argtypes = [ci]
            L.fs_kernel_name.restype = ctypes.c_char_p
            L.fs_version.argtypes = []
            L.fs_version.restype = ctypes.c_char_p
            _lib = L
    return _lib


def _ptr(buf) -> int:
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if hasattr(buf, "data_ptr"):
        return int(buf.data_ptr())
    if hasattr(buf, "ctypes"):
        return int(buf.ctypes.data)
    raise TypeError(f"cannot take the address of {type(buf)!r}")


def _stream(stream) -> int:
    if stream is None:
        return 0
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)          # torch.cuda.Stream


def _check(status: int, where: str) -> None:
    if status != FS_OK:
        raise FsError(status, where)


def fs_softmax(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """y = softmax(scale * x) over the last dimension of a [rows, cols] device tensor."""
    _check(lib().fs_softmax(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream)), "fs_softmax")


def fs_softmax_ex(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None,
                  kernel: int = FS_KERNEL_AUTO, threads: int = 0, cluster: int = 0) -> None:
    _check(lib().fs_softmax_ex(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream), kernel, threads, cluster),
           "fs_softmax_ex")


def fs_softmax_status(x, y, rows, cols, dtype, scale=1.0, stream=None, kernel=FS_KERNEL_AUTO, threads=0,
                      cluster=0) -> int:
    """fs_softmax_ex returning the raw status instead of raising (for error-path tests)."""
    return lib().fs_softmax_ex(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream), kernel, threads, cluster)


def fs_softmax_causal(x, y, rows: int, cols: int, q_offset: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """Causal softmax: row i keeps columns j <= i + q_offset; masked inputs are never read."""
    _check(lib().fs_softmax_causal(_ptr(x), _ptr(y), rows, cols, q_offset, dtype, scale, _stream(stream)),
           "fs_softmax_causal")


def fs_router_topk(x, w, idx, rows: int, cols: int, k: int, dtype: int, scale: float = 1.0, renormalize: bool = False,
                   stream=None) -> None:
    """Softmax over experts + top-k: w [rows, k] float32 and idx [rows, k] int32 device buffers."""
    _check(lib().fs_router_topk(_ptr(x), _ptr(w), _ptr(idx), rows, cols, k, dtype, scale, int(renormalize),
                                _stream(stream)), "fs_router_topk")


def fs_log_softmax(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """y = log_softmax(scale * x) over the last dimension of a [rows, cols] device tensor."""
    _check(lib().fs_log_softmax(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream)), "fs_log_softmax")


def fs_softmax_f32out(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """softmax(scale * x) of a bf16/fp16 [rows, cols] device tensor, written as float32."""
    _check(lib().fs_softmax_f32out(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream)), "fs_softmax_f32out")


def fs_softmax_masked(x, mask, y, rows: int, cols: int, q_rows: int, heads: int, dtype: int, scale: float = 1.0,
                      stream=None) -> None:
    """y = softmax(scale * x + mask): x rows ordered (batch, head, query), mask [batch * q_rows, cols] shared by the heads."""
    _check(lib().fs_softmax_masked(_ptr(x), _ptr(mask), _ptr(y), rows, cols, q_rows, heads, dtype, scale, _stream(stream)),
           "fs_softmax_masked")


def fs_softmax_backward(dy, y, dx, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """dx = scale * y * (dy - sum(dy * y)) over the last dimension: the gradient of softmax(scale * x)."""
    _check(lib().fs_softmax_backward(_ptr(dy), _ptr(y), _ptr(dx), rows, cols, dtype, scale, _stream(stream)),
           "fs_softmax_backward")


def fs_layer_norm(x, gamma, beta, y, rows: int, cols: int, dtype: int, eps: float = 1e-5, stream=None) -> None:
    """y = (x - mean) / sqrt(var + eps) * gamma + beta over the last dimension; gamma, beta may be None."""
    _check(lib().fs_layer_norm(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), rows, cols, dtype, eps, _stream(stream)),
           "fs_layer_norm")


def fs_group_norm(x, gamma, beta, y, n: int, channels: int, spatial: int, groups: int, dtype: int, eps: float = 1e-5,
                  stream=None) -> None:
    """Group normalisation of a dense [n, channels, spatial] tensor; gamma, beta per channel or None."""
    _check(lib().fs_group_norm(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), n, channels, spatial, groups, dtype, eps,
                               _stream(stream)), "fs_group_norm")


def fs_split_geometry(cols: int, dtype: int):
    """(cluster size, threads per block, slice bytes) of the split-row kernels for rows of `cols` elements, or None."""
    cs, t, sl = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int64(0)
    st = lib().fs_split_geometry(cols, dtype, ctypes.byref(cs), ctypes.byref(t), ctypes.byref(sl))
    if st == FS_ERR_UNSUPPORTED:
        return None
    _check(st, "fs_split_geometry")
    return cs.value, t.value, sl.value


def fs_select_kernel(rows: int, cols: int, dtype: int, x_align: int = 16, y_align: int = 16) -> int:
    return lib().fs_select_kernel(rows, cols, dtype, x_align, y_align)


def fs_softmax_host(x_host, y_host, rows: int, cols: int, dtype: int, scale: float = 1.0) -> None:
    _check(lib().fs_softmax_host(_ptr(x_host), _ptr(y_host), rows, cols, dtype, scale), "fs_softmax_host")


def fs_softmax_static(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None) -> None:
    """fs_softmax without any device allocation: status buffer and long-row scratch in a fixed device array."""
    _check(lib().fs_softmax_static(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream)), "fs_softmax_static")


def fs_static_status() -> int:
    """Reads and clears the status word of fs_softmax_static's fixed array (synchronises; allocates nothing)."""
    return lib().fs_static_status()


def fs_debug_checked_build() -> bool:
    """Whether the loaded library is the checked build (every global access range-checked)."""
    return bool(lib().fs_debug_checked_build())


def fs_debug_bad_address() -> int:
    """Checked build: the first address a kernel was refused since the last call (0 if none)."""
    a = ctypes.c_uint64(0)
    _check(lib().fs_debug_bad_address(ctypes.byref(a)), "fs_debug_bad_address")
    return int(a.value)


def fs_debug_shrink_writable(nbytes: int) -> None:
    """Checked build self-test: output ranges registered by this thread end `nbytes` early (0 restores)."""
    _check(lib().fs_debug_shrink_writable(nbytes), "fs_debug_shrink_writable")


def fs_debug_set_wait_polls(polls: int) -> None:
    """Poll cap of the bounded device-side waits on the current device (<= 0 restores the default)."""
    _check(lib().fs_debug_set_wait_polls(polls), "fs_debug_set_wait_polls")


def fs_debug_wait_probe(stream=None) -> None:
    """One block that waits for 16 bytes nobody copies: its bounded wait must run out."""
    _check(lib().fs_debug_wait_probe(_stream(stream)), "fs_debug_wait_probe")


def fs_debug_softmax_expire(x, y, rows: int, cols: int, dtype: int, scale: float = 1.0, stream=None, threads: int = 0,
                            cluster: int = 0) -> int:
    """The split-row kernel with every chunk barrier armed for 16 bytes too many; returns the raw status."""
    return lib().fs_debug_softmax_expire(_ptr(x), _ptr(y), rows, cols, dtype, scale, _stream(stream), threads, cluster)


def fs_copy(x, y, nbytes: int, stream=None) -> None:
    _check(lib().fs_copy(_ptr(x), _ptr(y), nbytes, _stream(stream)), "fs_copy")


def fs_device_status() -> int:
    return lib().fs_device_status()


def fs_release() -> None:
    _check(lib().fs_release(), "fs_release")


def fs_last_cuda_error() -> int:
    return lib().fs_last_cuda_error()


def fs_strerror(status: int) -> str:
    return lib().fs_strerror(status).decode()


def fs_kernel_name(kernel: int) -> str:
    return lib().fs_kernel_name(kernel).decode()


def fs_version() -> str:
    return lib().fs_version().decode()
