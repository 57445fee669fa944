"""Seeded synthetic inputs for the ESA select-plus-attend step.

This package only *draws inputs*: shapes, distributions and planted structure.
It performs none of the method's arithmetic (no compression of the step's
queries/keys, no scoring, no selection, no attention) and is the one module
that both the CPU oracle's tests and the CUDA path's tests/bench may import.
"""
from .configs import EsaShape, CONFIGS, get_config
from .generate import (
    to_bf16_bits,
    bf16_bits_to_f32,
    bf16_bits_to_f64,
    normal_bf16,
    compressor_weights,
    compressor_bias,
    qkv_rows,
    NeedlePlan,
    needle_plan,
)

__all__ = [
    "EsaShape", "CONFIGS", "get_config", "to_bf16_bits", "bf16_bits_to_f32",
    "bf16_bits_to_f64", "normal_bf16", "compressor_weights", "compressor_bias", "qkv_rows",
    "NeedlePlan", "needle_plan",
]
