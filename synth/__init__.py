"""Seeded synthetic MAR-shaped workloads (configs, weights, inputs, generation schedule).

This package only produces inputs.  It contains none of the method's arithmetic
(no LayerNorm, projection, attention, scoring or selection) so that the CPU
oracle and the CUDA path can both draw identical bytes from it without sharing
any computation.
"""
from .workload import (  # noqa: F401
    CONFIGS,
    MarConfig,
    BLOCK_FIELDS,
    mask_schedule,
    generation_orders,
    new_token_sets,
    make_weights,
    make_hidden,
    replacement_rows,
    round_to_bf16,
    peaked_weights,
    MAR_FIELDS,
    make_mar_weights,
    known_token_sets,
)
