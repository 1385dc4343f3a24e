"""Seeded synthetic gradient workloads.

This package only draws random arrays.  It holds none of the quantizer's
arithmetic, so both the CPU oracle's tests and the CUDA path's tests can feed
from it without sharing any of the method between them.
"""
from .generators import (  # noqa: F401
    Workload,
    WorkerSpec,
    tiny,
    dqsg_resnet18,
    ndqsg_resnet50,
    ndqsg_gpt2_small,
    sweep_point,
    by_name,
    with_dither_bits,
    WORKLOAD_NAMES,
)
