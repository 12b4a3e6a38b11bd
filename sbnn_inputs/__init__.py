"""Seeded synthetic inputs (tensors and group masks) shared by the tests and the benchmark.

This package draws numbers and index sets only.  It contains none of the
arithmetic of the convolution path and imports neither the CUDA library
nor the CPU oracle, so both can be fed the very same arrays.
"""
from .rng import uniform01, normal, u64_stream
from .masks import removed_units, group_mask_balanced, group_mask_layer_global, group_mask_magnitude, expand_mask, tap_pattern_mask, dw_pattern_mask
from .workloads import (
    single_conv_inputs,
    config5_family,
    mobilenet_v1_shapes,
    mobilenet_v1_inputs,
)

__all__ = [
    "uniform01", "normal", "u64_stream",
    "removed_units", "group_mask_balanced", "group_mask_layer_global",
    "group_mask_magnitude", "expand_mask", "tap_pattern_mask", "dw_pattern_mask",
    "single_conv_inputs", "config5_family", "mobilenet_v1_shapes", "mobilenet_v1_inputs",
]
