"""Seeded synthetic inputs for the Rollout-ResQ linear layer.

This package holds input generation only: shapes, seeds, value distributions and
the bf16 bit-pattern helpers.  It contains none of the method's arithmetic (no
quantizer, no mask, no product) and imports neither the CPU oracle nor the CUDA
library, so both can consume the same bit patterns.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    LayerSpec,
    WorkloadConfig,
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    make_activation,
    make_weight,
    make_layer,
)
