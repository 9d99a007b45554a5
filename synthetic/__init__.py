"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This package holds only counter-based pseudo-random generators.  It contains
none of the arithmetic of the sync step or of FedAvg and imports neither the
CUDA library nor the CPU oracle; both are fed from here so that they see the
same bits.
"""
from .gen import (  # noqa: F401
    KIND_GRAD, KIND_MASTER, KIND_SCALE, KIND_COUNT, KIND_MISC,
    stream_key, mix64_int, normal_fill_, normal_at, uniform_scale, sample_count,
    CONFIGS, config_by_name,
)
