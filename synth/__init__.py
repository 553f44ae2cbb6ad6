"""Seeded, addressable synthetic inputs shared by the oracle tests, the GPU parity
tests and the benchmark.

This package holds no attention or cache arithmetic: it only produces bf16 bit
patterns, head scores and head masks as functions of (seed, coordinates), so that
both the CPU oracle and the CUDA library can be fed the very same bytes, and so that
the history of a single (layer, batch row, KV head) can be regenerated on its own
without materialising a whole multi-gigabyte cache on the host.
"""
from .generator import (  # noqa: F401
    STREAM_K,
    STREAM_V,
    STREAM_Q,
    bf16_bits_to_float,
    head_mask,
    head_scores,
    normal_table,
    rows,
    unit_rows,
)
from .workloads import WORKLOADS, Workload, workload_mask  # noqa: F401
