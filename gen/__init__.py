"""Seeded synthetic inputs for the ToMA token-reduction path.

This module only draws numbers and lays them out; it contains none of the
method's arithmetic (no similarity, selection, softmax, merge or attention).
Both the CPU oracle's tests and the CUDA path's tests/benchmarks take their
inputs from here, so the two sides see identical arrays.
"""
from .inputs import (  # noqa: F401
    CONFIGS,
    TomaConfig,
    bf16_bits_to_f32,
    config,
    f32_to_bf16_bits,
    features,
    feature_sequence,
    neighbour_cosine,
    normal,
    round_to_dtype,
)
