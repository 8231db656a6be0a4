"""Seeded synthetic workloads for the ADSA decode-attention path.

This package holds only shapes and random-number plumbing: the five benchmark
configurations (LlamaGen-shaped attention stacks) and the counter-based
generators that turn a seed into bf16 q/k/v rows.  It contains none of the
method's arithmetic (no scoring, selection, softmax or cache logic), so both
the CPU oracle's tests and the CUDA path's tests can draw identical inputs
from it without sharing any code of the method itself.
"""
from .configs import CONFIGS, Workload, get_workload, pick_page_rows
from .gen import (
    bf16_bits_to_f32,
    f32_to_bf16_bits,
    late_state,
    layer_step_qkv,
    prefix_kv,
    structured_values,
)

__all__ = [
    "CONFIGS",
    "Workload",
    "get_workload",
    "pick_page_rows",
    "bf16_bits_to_f32",
    "f32_to_bf16_bits",
    "late_state",
    "layer_step_qkv",
    "prefix_kv",
    "structured_values",
]
