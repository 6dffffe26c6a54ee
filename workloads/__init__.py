"""Seeded synthetic workloads for the HMAR Markovian block-sparse attention path.

This package holds only shapes and random-number generation. It contains none of the
attention arithmetic, so both the CPU oracle's tests and the CUDA path's tests can draw
identical inputs from it without sharing any of the method's code.
"""
from .configs import CONFIGS, Workload, get_config  # noqa: F401
from .gen import (  # noqa: F401
    bf16_round,
    normal_tensor,
    scale_step_inputs,
    training_inputs,
)
