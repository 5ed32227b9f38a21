"""Helpers for the GPU parity tests: move stored bit patterns to the device, call the library
through its C ABI, and apply the oracle's comparator."""
import numpy as np
import torch

import paper_2607_24762_b200 as fs
from oracle import fso
from paper_2607_24762_b200 import workloads as W

GUARD = 64   # guard elements before and after every device buffer


def np_to_torch_bits(x: np.ndarray) -> torch.Tensor:
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16))
    return torch.from_numpy(x)


def torch_bits_to_np(t: torch.Tensor, dtype: int) -> np.ndarray:
    a = t.cpu().numpy()
    return a.view(np.uint16) if dtype != W.FP32 else a


def guard_pattern(n: int, np_dtype) -> np.ndarray:
    raw = (np.arange(n, dtype=np.uint32) * np.uint32(2654435761) >> np.uint32(7)).astype(np.uint16)
    if np_dtype == np.float32:
        return (raw.astype(np.uint32) | np.uint32(0x7F800000) | np.uint32(0x00400000)).view(np.float32)  # NaNs
    return raw | np.uint16(0x7FC0)


def run_softmax(x: np.ndarray, dtype: int, scale: float = 1.0, kernel: int = fs.FS_KERNEL_AUTO, threads: int = 0,
                cluster: int = 0, offset: int = 0, inplace: bool = False, stream=None, check_guards: bool = True,
                causal_q=None):
    """Runs the library on a copy of x placed `offset` elements past a 256-byte aligned address,
    with guard bands around input and output. Returns (status, y as stored numpy array or None)."""
    rows, cols = x.shape
    n = rows * cols
    st_dtype = W.NP_STORE[dtype]
    host = np.empty(GUARD + offset + n + GUARD, dtype=st_dtype)
    host[:GUARD + offset] = guard_pattern(GUARD + offset, st_dtype)
    host[GUARD + offset:GUARD + offset + n] = x.ravel()
    host[GUARD + offset + n:] = guard_pattern(GUARD, st_dtype)
    xd = np_to_torch_bits(host).cuda()
    if inplace:
        yd = xd
    else:
        yhost = np.empty_like(host)
        yhost[:] = guard_pattern(host.size, st_dtype)
        yd = np_to_torch_bits(yhost).cuda()
    esz = W.ELEM_SIZE[dtype]
    xp = xd.data_ptr() + (GUARD + offset) * esz
    yp = yd.data_ptr() + (GUARD + offset) * esz
    s = stream if stream is not None else torch.cuda.current_stream()
    if causal_q is None:
        status = fs.fs_softmax_status(xp, yp, rows, cols, dtype, scale, s, kernel, threads, cluster)
    else:
        status = fs.binding.lib().fs_softmax_causal(xp, yp, rows, cols, causal_q, dtype, scale, int(s.cuda_stream))
    torch.cuda.synchronize()
    if status != fs.FS_OK:
        return status, None
    out = torch_bits_to_np(yd, dtype)
    if check_guards:
        ref = host if inplace else yhost
        lo = slice(0, GUARD + offset)
        hi = slice(GUARD + offset + n, None)
        assert np.array_equal(out[lo].view(np.uint8), ref[lo].view(np.uint8)), "wrote before the output"
        assert np.array_equal(out[hi].view(np.uint8), ref[hi].view(np.uint8)), "wrote past the output"
        if not inplace:
            xin = torch_bits_to_np(xd, dtype)
            assert np.array_equal(xin.view(np.uint8), host.view(np.uint8)), "input was modified"
    return status, out[GUARD + offset:GUARD + offset + n].reshape(rows, cols).copy()


def check(x: np.ndarray, dtype: int, scale: float, y: np.ndarray):
    """Oracle comparison under the stated bar; returns the report."""
    want = fso.softmax_f64(x, dtype, scale)
    rep = fso.compare(y, dtype, want)
    assert rep.ok(dtype), rep
    return rep
