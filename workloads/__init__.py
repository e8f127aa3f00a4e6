"""Seeded synthetic inputs for the FBQuant inference linear.

This package only draws random tensors and rounds them to their storage
types.  It holds none of the layer's arithmetic (no packing, no dequantisation,
no contraction), so both the CPU oracle's tests and the CUDA path's tests can
share it without sharing any of the method.
"""
from .generators import (  # noqa: F401
    LinearInputs,
    LLAMA2_7B_SHAPES,
    LLAMA2_13B_SHAPES,
    bf16_bits_to_f64,
    f16_bits_to_f64,
    f32_to_bf16_bits,
    make_linear,
    make_exact_class,
    worked_example_e1,
)
