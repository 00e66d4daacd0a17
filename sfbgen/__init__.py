"""Seeded synthetic inputs for the sufficient-factor (SF) hot path.

This module only draws random tensors with the shapes, value distributions and
structure of the five workloads (MLR tiny / MLR large / DML / sparse-coding /
MLR at scale in bf16).  It contains none of the method's arithmetic: no
softmax, no hinge gate, no sufficient factor, no rank-K update.  Both the CPU
oracle's tests and the CUDA path's tests read their inputs from here, so the two
sides always see the same bytes.

Every tensor comes from its own counter-based Philox stream keyed by
(config index, tensor id, minibatch index), so any tensor can be regenerated
alone and in any order.
"""
from .configs import CONFIGS, scaled, get_config
from .generate import (
    make_inputs,
    batch_of,
    bf16_round_bits,
    bf16_bits_to_f32,
    philox,
)

__all__ = [
    "CONFIGS",
    "scaled",
    "get_config",
    "make_inputs",
    "batch_of",
    "bf16_round_bits",
    "bf16_bits_to_f32",
    "philox",
]
