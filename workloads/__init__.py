"""Seeded synthetic workloads: tensors, the five benchmark chain specs and the
random operator-DAG generator.

This package holds no operator arithmetic.  It only draws numbers from a
counter-based generator and writes operator-DAG spec text, so both the CUDA
library's tests and the CPU oracle can be fed from it without sharing any of
the method's code.
"""
from .tensors import uniform, normal, round_to_bf16_bits, bf16_bits_to_f32, make_tensor  # noqa: F401
from .configs import CONFIGS, get_config  # noqa: F401
