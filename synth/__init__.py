"""Seeded synthetic workload generators.

This package only draws random inputs (weights, prompts, KV contents) with the
shapes and value distributions of the benchmark configurations.  It holds none
of the method's arithmetic: no pruning, no coding, no model math.  Both the CPU
oracle's tests and the CUDA path's tests/bench take their inputs from here.
"""
from .workload import (  # noqa: F401
    ModelShape,
    TINY,
    LLAMA3_8B,
    QWEN_LARGE,
    llama_layer_shapes,
    student_t_weight,
    model_weights,
    random_prompt,
    kv_fill,
    activation_vector,
)
