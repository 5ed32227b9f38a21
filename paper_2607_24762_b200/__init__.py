"""libfsoftmax: last-dimension softmax for NVIDIA B200 (sm_100a) behind a C ABI.

``binding`` mirrors the C entry points of include/fsoftmax.h; ``workloads`` holds the seeded
synthetic inputs; ``_build`` compiles the shared library in-tree with nvcc.
"""
from .binding import (  # noqa: F401
    FS_DTYPE_BF16, FS_DTYPE_FP16, FS_DTYPE_FP32,
    FS_ERR_CUDA, FS_ERR_DEVICE_BOUNDS, FS_ERR_DEVICE_TIMEOUT, FS_ERR_INVALID_ARG, FS_ERR_UNSUPPORTED, FS_OK,
    FS_KERNEL_AUTO, FS_KERNEL_BLOCK, FS_KERNEL_BLOCK_TMA, FS_KERNEL_CLUSTER, FS_KERNEL_GENERIC, FS_KERNEL_WARP,
    FS_ROUTER_MAX_K, FS_STATIC_MAX_PAIRS, FS_STATIC_MAX_ROW_BYTES, FS_STATIC_SCRATCH_BYTES, KERNELS, FsError,
    fs_copy, fs_debug_bad_address, fs_debug_checked_build, fs_debug_set_wait_polls, fs_debug_shrink_writable, fs_debug_softmax_expire, fs_debug_wait_probe, fs_device_status, fs_group_norm, fs_kernel_name, fs_last_cuda_error, fs_layer_norm, fs_log_softmax, fs_release, fs_router_topk,
    fs_select_kernel, fs_split_geometry,
    fs_softmax, fs_softmax_backward, fs_softmax_causal, fs_softmax_ex, fs_softmax_f32out, fs_softmax_host, fs_softmax_masked, fs_softmax_static, fs_softmax_status, fs_static_status, fs_strerror, fs_version,
)
