"""Seeded synthetic inputs for the token-routing path.

This module only *draws inputs* (top-k expert ids, gate weights, hidden rows, source ranks
and an expert layout).  It holds none of the routing method's arithmetic, so both the CPU
oracle's tests and the CUDA path's tests/bench may feed from it without sharing any logic.
"""
from .configs import (  # noqa: F401
    BASE_SEED,
    CONFIG_NAMES,
    Workload,
    bf16_bits_from_f32,
    f32_from_bf16_bits,
    make_config,
    make_custom,
    make_layout,
    sample_gate_weights,
    sample_topk_ids,
)
