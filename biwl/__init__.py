"""Seeded synthetic workloads for batched discrete belief updates.

This package only draws inputs: generative-model arrays (A, B, D), observation
and action index streams, and the model description that goes with them.  It
holds none of the inference arithmetic, so both the CPU oracle's tests and the
CUDA path's tests can be fed from it without sharing any method code.
"""
from .configs import (  # noqa: F401
    Workload,
    make_config,
    make_sweep_config,
    make_model,
    sample_streams,
    SWEEP_SIZE,
    SWEEP_CAP_ENTRIES,
)
