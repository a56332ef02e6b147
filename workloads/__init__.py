"""Seeded synthetic inputs shaped like the five benchmark configurations.

This package serves both the CPU oracle's tests and the CUDA library's tests
and benchmark.  It holds none of the method's arithmetic (no paging, packing,
casting or assembly) and imports neither side.
"""
from .gen import (  # noqa: F401
    Workload, make_workload, CONFIG_NAMES, input_ids, span_values, embed_table, special_f32_bits,
    admit_free_schedule, span_grid, grad_values,
)
