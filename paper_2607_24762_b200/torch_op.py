"""Guarded PyTorch front end of libfsoftmax: the analogue of the paper's guarded dispatch
(Sec. III-E): per call, the library kernel runs only when it is available and compatible with the
call; every other call runs the unmodified eager operator, so a patched model keeps running in
eager mode and never sees a wrong or unsupported kernel.

    from paper_2607_24762_b200 import torch_op
    y = torch_op.softmax(x, dim=-1)                 # library kernel when the guard admits the call
    with torch_op.patched():                        # softmax, log_softmax, layer_norm, group_norm routed
        out = model(inputs)                         # through the guard for the duration of the block
    torch_op.stats()                                # how many calls went where, and why not

The guard admits a call when: the tensor is on a CUDA device, dtype fp32/bf16/fp16, the softmax
dimension is the last one (or the tensor can be seen that way without a copy), the tensor is
contiguous, no autograd graph is being recorded for it, and no output dtype conversion is asked
for other than eager attention's ``softmax(scores, dim=-1, dtype=torch.float32)`` on 16-bit scores
(which runs the library's 16-bit-in, float32-out kernel). log_softmax follows the same guard but
falls back for any ``dtype=``. This module is a convenience layer above the C ABI; the library
itself has no fallback.
"""
from __future__ import annotations

import contextlib
import threading
from collections import Counter

import torch

from . import binding

_DTYPES = {torch.float32: binding.FS_DTYPE_FP32, torch.bfloat16: binding.FS_DTYPE_BF16,
           torch.float16: binding.FS_DTYPE_FP16}
_stats = Counter()
_lock = threading.Lock()
_eager_softmax = torch.softmax            # the unpatched operators, captured at import
_eager_F_softmax = torch.nn.functional.softmax
_eager_T_softmax = torch.Tensor.softmax
_eager_log_softmax = torch.log_softmax
_eager_F_log_softmax = torch.nn.functional.log_softmax
_eager_F_layer_norm = torch.nn.functional.layer_norm
_eager_F_group_norm = torch.nn.functional.group_norm


def _count(key: str) -> None:
    with _lock:
        _stats[key] += 1


def stats(reset: bool = False) -> dict:
    """Calls per outcome: 'library', or 'eager:<reason>'."""
    with _lock:
        out = dict(_stats)
        if reset:
            _stats.clear()
    return out


def why_not(x: torch.Tensor, dim: int, dtype=None) -> str | None:
    """None when the guard admits the call, else the reason it goes to eager."""
    if not isinstance(x, torch.Tensor):
        return "not a tensor"
    if not x.is_cuda:
        return "not on a CUDA device"
    if x.dtype not in _DTYPES:
        return f"dtype {x.dtype}"
    if dtype is not None and dtype != x.dtype and not (dtype == torch.float32 and x.dtype in (torch.bfloat16, torch.float16)):
        return "output dtype conversion requested"
    if x.dim() == 0:
        return "0-d tensor"
    if dim not in (-1, x.dim() - 1):
        return "softmax dimension is not the last one"
    if not x.is_contiguous():
        return "not contiguous"
    if torch.is_grad_enabled() and x.requires_grad:
        return "autograd is recording"
    if x.numel() == 0:
        return "empty"
    return None


def softmax(x: torch.Tensor, dim: int = -1, dtype=None, scale: float = 1.0, out: torch.Tensor | None = None):
    """softmax(scale * x) over `dim`: the library kernel when admitted, else eager PyTorch."""
    reason = why_not(x, dim, dtype)
    if reason is None and out is not None and (out.shape != x.shape or out.dtype != x.dtype or
                                                not out.is_contiguous() or out.device != x.device):
        reason = "incompatible out tensor"
    if reason is None:
        try:
            binding.lib()
        except RuntimeError:
            reason = "library not built"
    if reason is not None:
        _count("eager:" + reason)
        xs = x if scale == 1.0 else x * scale
        y = _eager_softmax(xs, dim, dtype=dtype)
        if out is not None:
            out.copy_(y)
            return out
        return y
    cols = x.shape[-1]
    rows = x.numel() // cols
    if dtype == torch.float32 and x.dtype != torch.float32:
        # the eager-attention pattern softmax(scores, dim=-1, dtype=float32) on 16-bit scores
        if out is not None:
            _count("eager:out tensor with a dtype conversion")
            return out.copy_(_eager_softmax(x if scale == 1.0 else x * scale, dim, dtype=dtype))
        y = torch.empty(x.shape, dtype=torch.float32, device=x.device)
        with torch.cuda.device(x.device):
            binding.fs_softmax_f32out(x, y, rows, cols, _DTYPES[x.dtype], float(scale), torch.cuda.current_stream(x.device))
        _count("library")
        return y
    y = out if out is not None else torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_softmax(x, y, rows, cols, _DTYPES[x.dtype], float(scale), torch.cuda.current_stream(x.device))
    _count("library")
    return y


def log_softmax(x: torch.Tensor, dim: int = -1, dtype=None):
    """log_softmax over `dim`: the library kernel when admitted, else eager PyTorch."""
    reason = why_not(x, dim, dtype)
    if reason is None and dtype is not None and isinstance(x, torch.Tensor) and dtype != x.dtype:
        reason = "output dtype conversion requested"
    if reason is None:
        try:
            binding.lib()
        except RuntimeError:
            reason = "library not built"
    if reason is not None:
        _count("eager:" + reason)
        return _eager_log_softmax(x, dim, dtype=dtype)
    cols = x.shape[-1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_log_softmax(x, y, x.numel() // cols, cols, _DTYPES[x.dtype], 1.0, torch.cuda.current_stream(x.device))
    _count("library")
    return y


def _affine_ok(x, p, n):
    return p is None or (isinstance(p, torch.Tensor) and p.is_cuda and p.device == x.device and p.dtype == x.dtype and
                         p.is_contiguous() and p.numel() == n and not (torch.is_grad_enabled() and p.requires_grad))


def layer_norm(x: torch.Tensor, normalized_shape, weight=None, bias=None, eps: float = 1e-5):
    """layer_norm over the last dimension: the library kernel when admitted, else eager PyTorch."""
    shape = tuple(normalized_shape) if not isinstance(normalized_shape, int) else (normalized_shape,)
    reason = why_not(x, -1)
    if reason is None and (len(shape) != 1 or shape[0] != x.shape[-1]):
        reason = "normalized_shape is not the last dimension"
    if reason is None and not (_affine_ok(x, weight, x.shape[-1]) and _affine_ok(x, bias, x.shape[-1])):
        reason = "incompatible weight or bias"
    if reason is None:
        try:
            binding.lib()
        except RuntimeError:
            reason = "library not built"
    if reason is not None:
        _count("eager:" + reason)
        return _eager_F_layer_norm(x, shape, weight, bias, eps)
    cols = x.shape[-1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_layer_norm(x, weight, bias, y, x.numel() // cols, cols, _DTYPES[x.dtype], float(eps),
                              torch.cuda.current_stream(x.device))
    _count("library")
    return y


def group_norm(x: torch.Tensor, num_groups: int, weight=None, bias=None, eps: float = 1e-5):
    """group_norm of an [N, C, *] tensor: the library kernel when admitted, else eager PyTorch."""
    reason = why_not(x, -1)
    if reason is None and (x.dim() < 2 or num_groups < 1 or x.shape[1] % num_groups):
        reason = "shape"
    if reason is None and not (_affine_ok(x, weight, x.shape[1]) and _affine_ok(x, bias, x.shape[1])):
        reason = "incompatible weight or bias"
    if reason is None:
        try:
            binding.lib()
        except RuntimeError:
            reason = "library not built"
    if reason is not None:
        _count("eager:" + reason)
        return _eager_F_group_norm(x, num_groups, weight, bias, eps)
    n, ch = x.shape[0], x.shape[1]
    spatial = x.numel() // (n * ch)
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_group_norm(x, weight, bias, y, n, ch, spatial, num_groups, _DTYPES[x.dtype], float(eps),
                              torch.cuda.current_stream(x.device))
    _count("library")
    return y


def _patched_softmax(input, dim=None, *, dtype=None, **kw):        # torch.softmax(input, dim, dtype=None)
    if kw or dim is None:
        return _eager_softmax(input, dim, dtype=dtype, **kw)
    return softmax(input, dim, dtype)


def _patched_F_softmax(input, dim=None, _stacklevel=3, dtype=None):
    if dim is None:
        return _eager_F_softmax(input, dim, _stacklevel, dtype)
    return softmax(input, dim, dtype)


def _patched_T_softmax(self, dim=None, dtype=None, **kw):
    if kw or dim is None:
        return _eager_T_softmax(self, dim, dtype=dtype, **kw)
    return softmax(self, dim, dtype)


def _patched_F_log_softmax(input, dim=None, _stacklevel=3, dtype=None):
    if dim is None:
        return _eager_F_log_softmax(input, dim, _stacklevel, dtype)
    return log_softmax(input, dim, dtype)


def _patched_log_softmax(input, dim=None, *, dtype=None, **kw):
    if kw or dim is None:
        return _eager_log_softmax(input, dim, dtype=dtype, **kw)
    return log_softmax(input, dim, dtype)


@contextlib.contextmanager
def patched():
    """Route softmax, log_softmax, layer_norm and group_norm (torch.* and torch.nn.functional.*, and
    Tensor.softmax) through the guard for the duration of the block."""
    F = torch.nn.functional
    saved = (torch.softmax, F.softmax, torch.Tensor.softmax, torch.log_softmax, F.log_softmax, F.layer_norm, F.group_norm)
    torch.softmax = _patched_softmax
    F.softmax = _patched_F_softmax
    torch.Tensor.softmax = _patched_T_softmax
    torch.log_softmax = _patched_log_softmax
    F.log_softmax = _patched_F_log_softmax
    F.layer_norm = layer_norm
    F.group_norm = group_norm
    try:
        yield
    finally:
        (torch.softmax, F.softmax, torch.Tensor.softmax, torch.log_softmax, F.log_softmax, F.layer_norm, F.group_norm) = saved
