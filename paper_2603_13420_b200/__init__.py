"""Shared-prefix batched causal attention for B200 (sm_100a): Python face of libpskv.so.

``binding`` mirrors the C ABI in ``include/pskv.h``; ``inputs`` holds the seeded
synthetic workloads; ``build`` compiles the CUDA sources in-tree.
"""
from .binding import (  # noqa: F401
    PSKV_ERR_CUDA,
    PSKV_ERR_DEVICE_TIMEOUT,
    PSKV_ERR_INVALID_ARG,
    PSKV_ERR_UNSUPPORTED_ARCH,
    PSKV_ERR_UNSUPPORTED_SHAPE,
    PSKV_ERR_WORKSPACE,
    PSKV_OK,
    PskvError,
    pskv_attn_bwd,
    pskv_attn_bwd_decode,
    pskv_attn_bwd_decode_workspace_bytes,
    pskv_attn_bwd_multi,
    pskv_attn_bwd_multi_workspace_bytes,
    pskv_attn_bwd_static,
    pskv_attn_bwd_static_max_rows,
    pskv_attn_bwd_workspace_bytes,
    pskv_attn_fwd,
    pskv_attn_fwd_decode,
    pskv_attn_fwd_decode_workspace_bytes,
    pskv_attn_fwd_multi,
    pskv_attn_fwd_multi_workspace_bytes,
    pskv_attn_fwd_workspace_bytes,
    pskv_kernel_family,
    pskv_kernel_launches,
    pskv_kernel_timing_count,
    pskv_kernel_timing_enable,
    pskv_kernel_timing_name,
    pskv_kernel_timing_read,
    pskv_last_cuda_error,
    pskv_poll_device_status,
    pskv_status_string,
    pskv_version,
)
