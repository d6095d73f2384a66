"""Seeded synthetic workloads: layer tables shaped like the benchmark networks and
reproducible fp32 parameter / gradient values.

This module is input generation only.  It contains no part of the averaging
method (no norms, weights, averages or pulls) and is the one piece of code that
both the CPU oracle's tests and the GPU tests/bench are allowed to share.
"""
from .layer_tables import TABLES, layer_offsets, layer_sizes  # noqa: F401
from .values import CONFIGS, WorkloadConfig, make_inputs, philox_block, custom_config  # noqa: F401
