"""Seeded synthetic workloads: layer sets and gradient streams.

This package holds *inputs only*: shapes, hyper-parameters and the random
gradient streams.  None of the optimizer's arithmetic lives here, so both the
CPU oracle and the CUDA path may import it without sharing any method code.
"""
from .configs import LayerSpec, Workload, get_workload, WORKLOAD_NAMES  # noqa: F401
from .gradients import GradientStream, to_bf16_bits, bf16_bits_to_f32, initial_weight  # noqa: F401
