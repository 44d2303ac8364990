"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

This package holds NO arithmetic of the method (no block sums, no rounding of block sums,
no products): it only draws operands and gauge matrices.  Every value is a pure function
of (seed, tensor id, element index) through a counter-based generator, so the CPU oracle
and the CUDA path see the same bytes and nothing depends on a library RNG stream.
"""
from .generators import (  # noqa: F401
    normal, uniform, student_t3, activations_outlier, weights, integer_matrix, to_storage,
    gauge_cond_limited, gauge_log_uniform_cond, WORKLOADS,
)
