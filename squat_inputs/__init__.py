"""Seeded synthetic inputs for the SQuat KV-cache write path.

This package holds ONLY input generation: the five workload descriptions and the
counter-based generators that produce queries, keys and values for them.  It holds
none of the method's arithmetic, so both the CPU oracle's tests and the CUDA
library's tests / benchmark can draw identical bytes from it.
"""
from .configs import CONFIGS, WorkloadConfig, get_config
from .generators import (
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    gen_keys_unit,
    gen_queries_head,
    gen_values_unit,
    outlier_channels,
    gen_keys,
    gen_values,
    gen_queries,
    gen_start_block,
    round_to_dtype,
    to_f32,
)

__all__ = [
    "CONFIGS", "WorkloadConfig", "get_config",
    "bf16_bits_to_f32", "f32_to_bf16_bits", "round_to_dtype", "to_f32",
    "gen_keys_unit", "gen_values_unit", "gen_queries_head", "outlier_channels",
    "gen_keys", "gen_values", "gen_queries", "gen_start_block",
]
