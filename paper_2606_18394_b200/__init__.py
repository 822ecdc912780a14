"""B200-native tree-verification kernels (tree build, tree attention, acceptance, KV commit).

The product is ``libjet.so`` (C ABI declared in ``include/jet.h``); this package is the
thin ctypes binding with the same names.  Importing the package does not need a GPU;
calling an entry point needs the built library and fails loudly without it.
"""
from .binding import (  # noqa: F401
    JET_ERR_CUDA,
    JET_ERR_INVALID_ARG,
    JET_ERR_TIMEOUT,
    JET_ERR_UNSUPPORTED,
    JET_ERR_WORKSPACE,
    JET_ATTN_STABLE_PREFIX,
    JET_OK,
    JET_STATIC_ACCEPT_SCRATCH_BYTES,
    JetError,
    exported_symbols,
    jet_kv_compact,
    jet_kv_compact_tail,
    jet_tree_accept,
    jet_tree_accept_hidden,
    jet_tree_accept_hidden_workspace_bytes,
    jet_tree_accept_sample,
    jet_tree_accept_sample_workspace_bytes,
    jet_tree_accept_static,
    jet_tree_accept_workspace_bytes,
    jet_tree_build,
    jet_tree_build_logits,
    jet_tree_build_logits_workspace_bytes,
    jet_tree_build_scored,
    jet_tree_build_scored_workspace_bytes,
    jet_tree_build_workspace_bytes,
    jet_tree_verify_attn,
    jet_tree_verify_attn_ex,
    jet_tree_verify_attn_launches,
    jet_tree_verify_attn_plan,
    jet_tree_verify_attn_tail,
    jet_tree_verify_attn_tail_ex,
    jet_tree_verify_attn_workspace_bytes,
    load,
    status_string,
)
