"""Seeded synthetic inputs shared by the oracle tests, the GPU parity tests and
the benchmark.  This module holds no arithmetic of the method itself: it draws
random tensors of the workloads' shapes, rounds them to the storage types and
plants target arg-maxima on a path of a tree that the caller supplies.
"""
from .generators import (  # noqa: F401
    CONFIGS,
    bf16_bits_to_f32,
    binary_tree,
    chain_tree,
    f32_to_bf16_bits,
    make_attn_inputs,
    make_draft_logits,
    make_logp,
    make_paged_cache,
    make_target_logits,
    plant_path,
    random_tree,
    star_tree,
)
