"""Seeded synthetic inputs (model shapes, weights, prompts, references).

This package only *produces inputs*.  It holds none of the decoding method's
arithmetic and imports neither the CPU oracle nor the CUDA library, so that
both can be fed identical data without sharing code.
"""
from .generators import (  # noqa: F401
    ModelShape,
    SHAPES,
    bf16_bits_from_f32,
    f32_from_bf16_bits,
    make_prompt,
    make_weights,
    build_reference,
    weight_names,
)
