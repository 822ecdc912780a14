"""CPU oracle for the tree-verification hot path.

TEST INFRASTRUCTURE ONLY.  This package is the plain, slow, fp64 statement of
what the four operations compute, written from the paper's definitions.  It
shares no code with the CUDA path and must never be imported by the product
package: only the tests, the smoke check and the benchmark's CPU-baseline leg
may call it.
"""
from .jet_oracle import (  # noqa: F401
    anc_from_parent,
    bf16_bits_to_f64,
    depth_entropy_ref,
    gather_paged_prefix,
    kv_compact_ref,
    kv_compact_tail_ref,
    lm_head_argmax_ref,
    log_softmax_ref,
    target_probs_ref,
    tree_accept_ref,
    tree_accept_sample_ref,
    tree_attn_ref,
    tree_attn_rows_ref,
    tree_build_logits_ref,
    tree_build_ref,
)
