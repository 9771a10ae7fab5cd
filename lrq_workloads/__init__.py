"""Seeded synthetic inputs for the quantized-linear hot path.

This package only draws random arrays and converts number formats.  It holds none
of the method's arithmetic (no rotation, no quantizer, no contraction), so both the
CPU oracle's tests and the CUDA path's tests may feed from it without sharing any
computation.
"""
from .gen import (  # noqa: F401
    LayerSpec, CONFIGS, config_layers, make_weights, make_activations,
    make_orthogonal, f32_to_bf16_bits, bf16_bits_to_f32, bf16_bits_to_f64,
    default_clip_grid, salient_channels, make_block_rotations, make_staggered_permutation,
)
