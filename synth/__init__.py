"""Seeded synthetic inputs for the LBP-WHT linear-backward path.

This package holds input generation only: no Walsh-Hadamard arithmetic, no
matrix products, nothing the method computes.  Both the CPU oracle's tests and
the CUDA path's tests/benchmarks draw their tensors from here so that the two
sides see identical bits.
"""
from .inputs import (  # noqa: F401
    SEED,
    LayerCase,
    CONFIGS,
    config_cases,
    make_tensor,
    make_layer_inputs,
)
