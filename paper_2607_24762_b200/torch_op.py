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
contiguous, and no output dtype conversion is asked for other than eager attention's
``softmax(scores, dim=-1, dtype=torch.float32)`` on 16-bit scores (which runs the library's
16-bit-in, float32-out kernel). log_softmax follows the same guard but falls back for any ``dtype=``.

The admitted calls go through operators registered with ``torch.library`` under the namespace
``fsoftmax`` -- ``torch.ops.fsoftmax.softmax(x, scale)``, ``softmax_backward(dy, y, scale)``,
``log_softmax(x)``, ``layer_norm(x, weight, bias, eps)``, ``group_norm(x, groups, weight, bias, eps)`` -- each
with a fake (meta) implementation, so that a traced or compiled model carries them as opaque nodes,
and softmax with an autograd formula that runs the library's backward kernel: a softmax whose input
requires grad stays on the library in both directions. The other three have no backward kernel, so
the guard sends them to eager while autograd is recording. Each operator applies the guard again on
the tensors it is handed (a compiled graph may call it directly) and computes the same result with
eager PyTorch when the guard refuses. This module is a convenience layer above the C ABI; the
library itself has no fallback.
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


def why_not(x: torch.Tensor, dim: int, dtype=None, grad_ok: bool = False) -> str | None:
    """None when the guard admits the call, else the reason it goes to eager. `grad_ok`: the operator has
    an autograd formula, so an input that requires grad is no reason to refuse."""
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
    if not grad_ok and torch.is_grad_enabled() and x.requires_grad:
        return "autograd is recording"
    if x.numel() == 0:
        return "empty"
    return None


# ---------------------------------------------------------------------------------------------
# operators registered with torch.library (namespace "fsoftmax")
# ---------------------------------------------------------------------------------------------

def _library_ok(x: torch.Tensor, *others) -> bool:
    """The guard as the operators apply it to the tensors they are handed."""
    if why_not(x, -1, grad_ok=True) is not None:
        return False
    for t in others:
        if t is not None and not (t.is_cuda and t.device == x.device and t.dtype == x.dtype and t.is_contiguous()):
            return False
    try:
        binding.lib()
    except RuntimeError:
        return False
    return True


@torch.library.custom_op("fsoftmax::softmax", mutates_args=())
def _op_softmax(x: torch.Tensor, scale: float) -> torch.Tensor:
    if not _library_ok(x):
        _count("eager:operator called on tensors the guard refuses")
        return _eager_softmax(x if scale == 1.0 else x * scale, -1)
    cols = x.shape[-1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_softmax(x, y, x.numel() // cols, cols, _DTYPES[x.dtype], scale, torch.cuda.current_stream(x.device))
    _count("library")
    return y


@_op_softmax.register_fake
def _(x, scale):
    return torch.empty_like(x)


@torch.library.custom_op("fsoftmax::softmax_backward", mutates_args=())
def _op_softmax_backward(dy: torch.Tensor, y: torch.Tensor, scale: float) -> torch.Tensor:
    """dx = scale * y * (dy - sum(dy * y)) over the last dimension."""
    if dy.shape != y.shape or not _library_ok(y, dy) or dy.dtype != y.dtype:
        _count("eager:operator called on tensors the guard refuses")
        return (scale * y * (dy - (dy * y).sum(dim=-1, keepdim=True))).to(y.dtype)
    cols = y.shape[-1]
    dx = torch.empty_like(y)
    with torch.cuda.device(y.device):
        binding.fs_softmax_backward(dy, y, dx, y.numel() // cols, cols, _DTYPES[y.dtype], scale,
                                    torch.cuda.current_stream(y.device))
    _count("library")
    return dx


@_op_softmax_backward.register_fake
def _(dy, y, scale):
    return torch.empty_like(y)


def _softmax_setup_context(ctx, inputs, output):
    ctx.save_for_backward(output)
    ctx.scale = inputs[1]


def _softmax_autograd(ctx, grad):
    (y,) = ctx.saved_tensors
    return torch.ops.fsoftmax.softmax_backward(grad.contiguous(), y, ctx.scale), None


torch.library.register_autograd("fsoftmax::softmax", _softmax_autograd, setup_context=_softmax_setup_context)


@torch.library.custom_op("fsoftmax::log_softmax", mutates_args=())
def _op_log_softmax(x: torch.Tensor) -> torch.Tensor:
    if not _library_ok(x):
        _count("eager:operator called on tensors the guard refuses")
        return _eager_log_softmax(x, -1)
    cols = x.shape[-1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_log_softmax(x, y, x.numel() // cols, cols, _DTYPES[x.dtype], 1.0, torch.cuda.current_stream(x.device))
    _count("library")
    return y


@_op_log_softmax.register_fake
def _(x):
    return torch.empty_like(x)


@torch.library.custom_op("fsoftmax::layer_norm", mutates_args=())
def _op_layer_norm(x: torch.Tensor, weight: torch.Tensor | None, bias: torch.Tensor | None, eps: float) -> torch.Tensor:
    if not _library_ok(x, weight, bias):
        _count("eager:operator called on tensors the guard refuses")
        return _eager_F_layer_norm(x, (x.shape[-1],), weight, bias, eps)
    cols = x.shape[-1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_layer_norm(x, weight, bias, y, x.numel() // cols, cols, _DTYPES[x.dtype], eps,
                              torch.cuda.current_stream(x.device))
    _count("library")
    return y


@_op_layer_norm.register_fake
def _(x, weight, bias, eps):
    return torch.empty_like(x)


@torch.library.custom_op("fsoftmax::group_norm", mutates_args=())
def _op_group_norm(x: torch.Tensor, groups: int, weight: torch.Tensor | None, bias: torch.Tensor | None,
                   eps: float) -> torch.Tensor:
    if x.dim() < 2 or not _library_ok(x, weight, bias):
        _count("eager:operator called on tensors the guard refuses")
        return _eager_F_group_norm(x, groups, weight, bias, eps)
    n, ch = x.shape[0], x.shape[1]
    y = torch.empty_like(x)
    with torch.cuda.device(x.device):
        binding.fs_group_norm(x, weight, bias, y, n, ch, x.numel() // (n * ch), groups, _DTYPES[x.dtype], eps,
                              torch.cuda.current_stream(x.device))
    _count("library")
    return y


@_op_group_norm.register_fake
def _(x, groups, weight, bias, eps):
    return torch.empty_like(x)


# ---------------------------------------------------------------------------------------------
# the guarded front end
# ---------------------------------------------------------------------------------------------

def softmax(x: torch.Tensor, dim: int = -1, dtype=None, scale: float = 1.0, out: torch.Tensor | None = None):
    """softmax(scale * x) over `dim`: the library kernel when admitted, else eager PyTorch."""
    plain = out is None and (dtype is None or (isinstance(x, torch.Tensor) and dtype == x.dtype))
    reason = why_not(x, dim, dtype, grad_ok=plain)
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
    if out is None:
        return torch.ops.fsoftmax.softmax(x, float(scale))          # registered operator: autograd, fake tensors
    with torch.cuda.device(x.device):
        binding.fs_softmax(x, out, rows, cols, _DTYPES[x.dtype], float(scale), torch.cuda.current_stream(x.device))
    _count("library")
    return out


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
    return torch.ops.fsoftmax.log_softmax(x)


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
    return torch.ops.fsoftmax.layer_norm(x, weight, bias, float(eps))


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
    return torch.ops.fsoftmax.group_norm(x, int(num_groups), weight, bias, float(eps))


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
