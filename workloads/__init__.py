"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle drivers.

This package draws random numbers and shapes them like the workloads; it contains none of the
method's arithmetic (no attention, no scoring, no selection).
"""
from .gen import (  # noqa: F401
    CONFIGS,
    WorkloadConfig,
    get_config,
    make_rng,
    to_cache_dtype,
    prompt_kv,
    DecodeStream,
)
