"""Seeded synthetic workloads for the LASER STA+GSTA forward pass.

This package only draws random inputs (item / candidate embeddings, ragged
lengths, projection weights) with the shapes and value distributions of the
benchmark configurations.  It contains none of the method's arithmetic and is
the single module shared by the CPU oracle's tests and the CUDA path's tests
and benchmark.
"""
from .configs import (  # noqa: F401
    CONFIGS,
    Workload,
    WorkloadSpec,
    make_workload,
    make_custom,
    make_ffn_weights,
    make_gsta_inputs,
    round_to_dtype,
)
