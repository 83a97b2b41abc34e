"""Seeded synthetic inputs for the W4A4 + low-rank linear layer.

This package only *produces inputs* (activations, smoothing vector, low-rank
factors, residual codes with their group scales, bias, clip table).  It holds
none of the forward path's arithmetic and is the one module that both the CPU
oracle's tests and the CUDA path's tests / benchmark may import.
"""
from .generator import (  # noqa: F401
    LayerInputs,
    bf16_bits,
    bf16_to_f32,
    make_activations,
    make_clip_table,
    make_layer_direct,
    make_layer_svd,
    CONFIG_SHAPES,
)
