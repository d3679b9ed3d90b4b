"""Seeded synthetic workloads shared by the tests, the smoke check and the benchmark.

This package only draws random tensors with the shapes and value structure of the workloads;
it contains none of the method's arithmetic and imports neither the oracle nor the CUDA path.
"""
from .configs import WorkloadConfig, CONFIGS, get_config  # noqa: F401
from .generate import generate_layer, generate_model, to_numpy64  # noqa: F401
