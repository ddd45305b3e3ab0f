"""Seeded synthetic inputs and workload shapes.

This module serves both the CPU oracle's tests and the CUDA library's tests and
benchmark.  It holds shapes and random-number recipes only, none of the
method's arithmetic (no quantiser, no initialisation of s and z, no packing).
"""
from .configs import LINEARS, CONFIGS, Linear, Config, get_config  # noqa: F401
from .generators import (  # noqa: F401
    BASE_SEED, tensor_seed, normal_bf16, student_t_bf16, weight_for, activations_for,
    to_bf16_bits, from_bf16_bits,
)
