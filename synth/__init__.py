"""Seeded synthetic inputs for the bounded-cache MoE decode step.

This module only manufactures bytes: Gaussian weight tensors and AR(1) hidden-state
streams, keyed by (seed, tensor id) through a counter-based generator (numpy's Philox).
It holds none of the method's arithmetic (no routing, no softmax, no cache, no FFN),
so both the CPU oracle's tests and the CUDA library's callers may use it; neither of
those two imports the other.
"""
from .workloads import (  # noqa: F401
    Shape,
    CONFIGS,
    config,
    expert_block_elems,
    expert_block_bytes,
    bf16_round_to_bits,
    bf16_bits_to_f32,
    fp8_e4m3_round_to_bits,
    fp8_e4m3_bits_to_f32,
    int4_g32_encode,
    int4_g32_decode,
    INT4_GROUP,
    widen,
    FP8_SHIFT,
    gen_router,
    gen_shared_gate,
    gen_expert_block,
    gen_shared_block,
    fill_expert_store,
    expert_matrices,
    HiddenStream,
)
