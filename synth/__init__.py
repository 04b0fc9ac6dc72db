"""Seeded synthetic inputs for the CollectiveKV decode path.

This package only draws random tensors of the right shapes; it holds none of
the method's arithmetic (no gather, no concat, no attention).  It is the one
module both the CPU oracle's tests and the CUDA path's tests/bench may import.
"""
from .workloads import (  # noqa: F401
    WORKLOADS,
    Workload,
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    generate,
    scaled,
)
