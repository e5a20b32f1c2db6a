"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This package only *draws* arrays (model weights as bf16 bit patterns, context
token arrays) and names the workload configurations.  It contains none of the
method's arithmetic: no transformer op, no matcher, no acceptance logic.
"""
from .configs import ModelConfig, CONFIGS, get_config
from .generate import (LayerWeights, ModelWeights, make_weights, make_context,
                       f32_to_bf16_bits, bf16_bits_to_f32)

__all__ = ["ModelConfig", "CONFIGS", "get_config", "LayerWeights", "ModelWeights",
           "make_weights", "make_context", "f32_to_bf16_bits", "bf16_bits_to_f32"]
