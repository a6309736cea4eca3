"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package only *makes data*: counter-based random numbers, planted structure and
bf16 rounding.  It contains none of the method's arithmetic (no attention, no probe,
no selection, no routing) and imports neither the oracle nor the CUDA binding.
"""
from .generator import (  # noqa: F401
    LayerSpec,
    SegmentSpec,
    bf16_bits_to_f32,
    bf16_bits_to_f64,
    config1_spec,
    config2_spec,
    config3_spec,
    config4_layer_spec,
    f32_to_bf16_bits,
    fixed_routes_config2,
    make_layer,
    tiny_spec,
)
