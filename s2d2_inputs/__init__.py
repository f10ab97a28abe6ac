"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This package holds model shapes, random-init weights, prompts and nothing of
the decoding method's arithmetic: no softmax, no acceptance rule, no random
uniforms of the method.  Both sides draw their inputs from here so that they
see identical bytes.
"""
from .configs import CONFIGS, ModelConfig, WorkloadConfig, get_config  # noqa: F401
from .generate import (  # noqa: F401
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    generate_prompts,
    generate_weights,
    weight_shapes,
)
