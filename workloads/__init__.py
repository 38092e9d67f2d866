"""Seeded synthetic inputs for the five composed-module workloads.

This package holds storage-format code only (random draws, bf16 rounding,
layout permutations).  None of the operators' arithmetic lives here: it is the
one module that both the CPU oracle's tests and the CUDA path's tests read, so
that the two sides consume exactly the same bytes.
"""
from .generate import (  # noqa: F401
    Tensor,
    bf16_bits_to_f64,
    c1,
    c2,
    c3,
    c4,
    c5,
    c6,
    c7,
    c8,
    c9,
    e4m3_bits_to_f64,
    f32_to_e4m3_bits,
    f32_to_bf16_bits,
    int_valued,
    make,
)
