"""Dithered (DQSG) and nested dithered (NDQSG) gradient quantization on NVIDIA B200.

Thin Python binding over the C ABI in ``include/dq.h``; every step of the path runs in the CUDA
kernels of ``csrc/``.  PyTorch is used for device memory and streams only.
"""
from .binding import (  # noqa: F401
    DQ_KIND_DQSG,
    DQ_KIND_NDQSG,
    DQ_WARN_NONFINITE_SCALE,
    DQ_ERR_COPY_TIMEOUT,
    DqError,
    DqParams,
    DqMsg,
    Message,
    lib,
    packed_words,
    num_buckets,
    default_levels,
    status_string,
    dqsg_encode,
    ndqsg_encode,
    dqsg_decode_aggregate,
    ndqsg_decode_aggregate,
    ndqsg_decode_aggregate_running,
    dqsg_decode_aggregate_half_dithered,
    code_histogram,
    entropy_bits_per_element,
    encode_workspace_bytes,
    decode_workspace_bytes,
    dqsg_encode_host,
    ndqsg_encode_host,
    ndqsg_decode_aggregate_host,
    dqsg_encode_host_static,
    STATIC_SCRATCH_BYTES,
    device_error_flags,
    launch_count,
)
