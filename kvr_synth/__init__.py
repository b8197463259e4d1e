"""Seeded synthetic inputs for the paged-KV suspend/resume path.

This module only draws numbers: geometries, block-id permutations, context
lengths, wait times and KV bytes.  It contains none of the arithmetic of the
data path itself (no gather, scatter, allocation or admission rule), so both
the CPU oracle's tests and the CUDA library's tests may take inputs from it.
"""
from .gen import (  # noqa: F401
    CONFIGS, Workload, bf16_normal_bits, context_lengths, event_trace, fill_bytes,
    free_order, occupancy_fillers, paper_wait_family, poisson_arrivals, wait_mixture,
)
