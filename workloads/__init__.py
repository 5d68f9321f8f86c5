"""Seeded synthetic inputs for the codebook-binary linear layer.

This package only draws numbers and lays them out; it holds none of the
method's arithmetic (no packing, no decode, no dot products).  Both the CPU
oracle's tests and the CUDA path's tests/bench feed from here, so the two
sides see the same bytes.
"""
from .gen import (  # noqa: F401
    LayerSpec,
    LayerData,
    CONFIGS,
    config_layers,
    make_layer,
    make_codebook_pm1,
    make_indices,
    make_sign_words,
    make_alpha_f16,
    make_x,
    f32_to_bf16_bits,
    bf16_bits_to_f32,
    stream_seed,
)
