"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests/bench.

This module holds input *generation* only: model shapes, random weights rounded once to
bfloat16, token ids, physical block-id permutations and the counter-based byte pattern used
to fill paged caches.  None of the method's arithmetic (norms, projections, attention,
pack/unpack) lives here, so the oracle and the CUDA path can both consume it without
sharing any computation.
"""
from .configs import ModelShape, SHAPES, kv_page_bytes
from .inputs import (bf16_round_f32, f32_to_bf16_bits, bf16_bits_to_f32, layer_weights,
                     head_weights, token_ids, block_permutation, pattern_bytes,
                     PATTERN_MUL, STRESS_BLOCK_COUNTS)

__all__ = [
    "ModelShape", "SHAPES", "kv_page_bytes", "bf16_round_f32", "f32_to_bf16_bits",
    "bf16_bits_to_f32", "layer_weights", "head_weights", "token_ids", "block_permutation",
    "pattern_bytes", "PATTERN_MUL", "STRESS_BLOCK_COUNTS",
]
