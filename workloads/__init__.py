"""Seeded synthetic workloads for the ADORE decode path.

This package only describes shapes and draws random numbers. It contains none of the
method's arithmetic (no attention, controller, selection, projection or RoPE), so that
the CPU oracle and the CUDA library can both be fed from it without sharing any code
that could hide a common mistake.
"""
from .configs import WorkloadConfig, CONFIGS, get_config, sweep_points  # noqa: F401
from .generate import (  # noqa: F401
    substream,
    round_to_dtype,
    controller_weights,
    hidden_rows,
    projection_weights,
    query_weights,
    gaussian,
    rebuild_flags,
    slot_weights,
)
