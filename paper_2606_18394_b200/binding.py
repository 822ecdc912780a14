"""ctypes binding of libjet.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors used purely as device-memory handles (``data_ptr()``); every
step of the path runs inside the library's kernels.  There is no fallback: if the shared
library is missing the import of any entry point raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libjet.so")

JET_OK = 0
JET_ERR_INVALID_ARG = -1
JET_ERR_UNSUPPORTED = -2
JET_ERR_WORKSPACE = -3
JET_ERR_CUDA = -4
JET_ERR_TIMEOUT = -5
JET_ATTN_STABLE_PREFIX = 1                     # jet.h: flag of the *_ex attention calls
JET_STATIC_ACCEPT_SCRATCH_BYTES = 1 << 20     # jet.h: built-in scratch of jet_tree_accept_static

_c = ctypes
_vp, _i, _i64, _f, _sz = _c.c_void_p, _c.c_int, _c.c_int64, _c.c_float, _c.c_size_t

_SIGNATURES = {
    "jet_status_string": (_c.c_char_p, [_c.c_int32]),
    "jet_tree_build_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "jet_tree_build": (_c.c_int32, [_vp, _i64, _i64, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp,
                                    _vp, _vp, _sz, _vp]),
    "jet_tree_build_scored_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "jet_tree_build_scored": (_c.c_int32, [_vp, _i64, _i64, _vp, _i, _i, _i, _i, _i, _vp, _i, _f, _vp, _vp, _vp, _vp,
                                           _vp, _vp, _vp, _vp, _sz, _vp]),
    "jet_tree_build_logits_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "jet_tree_build_logits": (_c.c_int32, [_vp, _i64, _i64, _vp, _i, _i, _i, _i, _i, _vp, _i, _f, _vp, _vp, _vp, _vp,
                                           _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "jet_tree_verify_attn_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "jet_tree_verify_attn_launches": (_i, [_i, _i, _i, _i, _i, _i]),
    "jet_tree_verify_attn_plan": (_i, [_i, _i, _i, _i, _i, _i, _vp]),
    "jet_tree_verify_attn": (_c.c_int32, [_vp, _vp, _vp, _vp, _i, _i, _i64, _vp, _i, _vp, _vp, _vp, _vp,
                                          _i, _i, _i, _i, _i, _i64, _f, _vp, _vp, _vp, _vp, _sz, _vp]),
    "jet_tree_verify_attn_tail": (_c.c_int32, [_vp, _vp, _vp, _vp, _i, _i, _i64, _vp, _i, _vp, _vp,
                                               _i, _i, _i, _i, _i, _i64, _f, _vp, _vp, _vp, _vp, _sz, _vp]),
    "jet_tree_verify_attn_ex": (_c.c_int32, [_vp, _vp, _vp, _vp, _i, _i, _i64, _vp, _i, _vp, _vp, _vp, _vp,
                                             _i, _i, _i, _i, _i, _i64, _f, _vp, _vp, _vp, _vp, _sz, _vp,
                                             _c.c_uint32]),
    "jet_tree_verify_attn_tail_ex": (_c.c_int32, [_vp, _vp, _vp, _vp, _i, _i, _i64, _vp, _i, _vp, _vp,
                                                  _i, _i, _i, _i, _i, _i64, _f, _vp, _vp, _vp, _vp, _sz, _vp,
                                                  _c.c_uint32]),
    "jet_kv_compact_tail": (_c.c_int32, [_vp, _vp, _i64, _i64, _vp, _i, _i, _vp, _vp, _vp, _i, _i, _i, _i,
                                         _i, _i, _vp]),
    "jet_tree_accept_workspace_bytes": (_sz, [_i, _i, _i]),
    "jet_tree_accept": (_c.c_int32, [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp,
                                     _vp, _vp, _sz, _vp]),
    "jet_tree_accept_hidden_workspace_bytes": (_sz, [_i, _i]),
    "jet_tree_accept_hidden": (_c.c_int32, [_vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp,
                                            _vp, _vp, _sz, _vp]),
    "jet_tree_accept_static": (_c.c_int32, [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp,
                                            _vp, _vp]),
    "jet_tree_accept_sample_workspace_bytes": (_sz, [_i, _i, _i]),
    "jet_tree_accept_sample": (_c.c_int32, [_vp, _i64, _f, _vp, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                            _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "jet_kv_compact": (_c.c_int32, [_vp, _vp, _vp, _vp, _i64, _i64, _vp, _i, _i, _vp, _vp, _vp, _i, _i,
                                    _i, _i, _i, _i, _vp]),
}

_lib = None


class JetError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def load():
    """Load libjet.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2606_18394_b200.build`; "
                "there is no fallback path")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def exported_symbols():
    return sorted(_SIGNATURES)


def _p(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(status: int, where: str):
    if status != JET_OK:
        raise JetError(status, where)


def status_string(status: int) -> str:
    return load().jet_status_string(status).decode()


def jet_tree_build_workspace_bytes(batch, N, V, W) -> int:
    return load().jet_tree_build_workspace_bytes(batch, N, V, W)


def jet_tree_build(logp, root_token, batch, N, V, W, B, parent, depth, token, score, anc_mask, n_nodes,
                   workspace, workspace_bytes=None, logp_batch_stride=None, logp_depth_stride=None,
                   stream=None, check=True):
    bs = logp_batch_stride if logp_batch_stride is not None else logp.stride(0)
    ds = logp_depth_stride if logp_depth_stride is not None else logp.stride(1)
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_build(_p(logp), bs, ds, _p(root_token), batch, N, V, W, B, _p(parent), _p(depth),
                               _p(token), _p(score), _p(anc_mask), _p(n_nodes), _p(workspace), wb,
                               _stream(stream))
    if check:
        _check(st, "jet_tree_build")
    return st


SCORE_ACCUM_LOGP, SCORE_ENTROPY, SCORE_HYBRID = 0, 1, 2


def jet_tree_build_scored_workspace_bytes(batch, N, V, W) -> int:
    return load().jet_tree_build_scored_workspace_bytes(batch, N, V, W)


def jet_tree_build_scored(logp, root_token, batch, N, V, W, B, score_mode, alpha, parent, depth, token, score,
                          anc_mask, n_nodes, depth_entropy, workspace, workspace_bytes=None,
                          logp_batch_stride=None, logp_depth_stride=None, stream=None, check=True,
                          node_budget=None):
    bs = logp_batch_stride if logp_batch_stride is not None else logp.stride(0)
    ds = logp_depth_stride if logp_depth_stride is not None else logp.stride(1)
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_build_scored(_p(logp), bs, ds, _p(root_token), batch, N, V, W, B, _p(node_budget),
                                      int(score_mode), float(alpha), _p(parent), _p(depth), _p(token), _p(score), _p(anc_mask),
                                      _p(n_nodes), _p(depth_entropy), _p(workspace), wb, _stream(stream))
    if check:
        _check(st, "jet_tree_build_scored")
    return st


def jet_tree_build_logits_workspace_bytes(batch, N, V, W) -> int:
    return load().jet_tree_build_logits_workspace_bytes(batch, N, V, W)


def jet_tree_build_logits(logits, root_token, batch, N, V, W, B, score_mode, alpha, parent, depth, token, score,
                          anc_mask, n_nodes, depth_entropy, depth_lse, workspace, workspace_bytes=None,
                          logits_batch_stride=None, logits_depth_stride=None, stream=None, check=True,
                          node_budget=None):
    bs = logits_batch_stride if logits_batch_stride is not None else logits.stride(0)
    ds = logits_depth_stride if logits_depth_stride is not None else logits.stride(1)
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_build_logits(_p(logits), bs, ds, _p(root_token), batch, N, V, W, B, _p(node_budget),
                                      int(score_mode), float(alpha), _p(parent), _p(depth), _p(token), _p(score),
                                      _p(anc_mask), _p(n_nodes), _p(depth_entropy), _p(depth_lse), _p(workspace), wb,
                                      _stream(stream))
    if check:
        _check(st, "jet_tree_build_logits")
    return st


def jet_tree_verify_attn_workspace_bytes(batch, B, Hq, Hkv, D, max_seq_len) -> int:
    return load().jet_tree_verify_attn_workspace_bytes(batch, B, Hq, Hkv, D, max_seq_len)


def jet_tree_verify_attn_launches(batch, B, Hq, Hkv, D, max_seq_len) -> int:
    return load().jet_tree_verify_attn_launches(batch, B, Hq, Hkv, D, max_seq_len)


def jet_tree_verify_attn_plan(batch, B, Hq, Hkv, D, max_seq_len) -> dict:
    """The launch plan of a shape: query tiles per CTA, tile groups, key slices, merge form, CTA pairs."""
    out = (_c.c_int32 * 5)()
    if not load().jet_tree_verify_attn_plan(batch, B, Hq, Hkv, D, max_seq_len, _c.cast(out, _c.c_void_p)):
        raise JetError(JET_ERR_INVALID_ARG, "jet_tree_verify_attn_plan")
    forms = {0: "none", 1: "cluster", 2: "workspace", 3: "second launch"}
    return dict(query_tiles_per_cta=out[0], tile_groups=out[1], key_slices=out[2], merge=forms[out[3]], pair=bool(out[4]))


def jet_tree_verify_attn(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len,
                         max_seq_len, tree_k, tree_v, anc_mask, n_nodes, batch, B, Hq, Hkv, D,
                         kv_batch_stride, softmax_scale, out, lse, device_status, workspace,
                         workspace_bytes=None, stream=None, check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_verify_attn(_p(q), _p(k_cache), _p(v_cache), _p(page_table), max_pages_per_seq,
                                     page_size, num_pages, _p(seq_len), max_seq_len, _p(tree_k), _p(tree_v),
                                     _p(anc_mask), _p(n_nodes), batch, B, Hq, Hkv, D, kv_batch_stride,
                                     softmax_scale, _p(out), _p(lse), _p(device_status), _p(workspace), wb,
                                     _stream(stream))
    if check:
        _check(st, "jet_tree_verify_attn")
    return st


def jet_tree_verify_attn_tail(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len,
                              max_seq_len, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride,
                              softmax_scale, out, lse, device_status, workspace, workspace_bytes=None, stream=None,
                              check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_verify_attn_tail(_p(q), _p(k_cache), _p(v_cache), _p(page_table), max_pages_per_seq,
                                          page_size, num_pages, _p(seq_len), max_seq_len, _p(anc_mask),
                                          _p(n_nodes), batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                                          _p(out), _p(lse), _p(device_status), _p(workspace), wb, _stream(stream))
    if check:
        _check(st, "jet_tree_verify_attn_tail")
    return st


def jet_tree_verify_attn_ex(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages, seq_len,
                            max_seq_len, tree_k, tree_v, anc_mask, n_nodes, batch, B, Hq, Hkv, D,
                            kv_batch_stride, softmax_scale, out, lse, device_status, workspace, flags,
                            workspace_bytes=None, stream=None, check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_verify_attn_ex(_p(q), _p(k_cache), _p(v_cache), _p(page_table), max_pages_per_seq,
                                        page_size, num_pages, _p(seq_len), max_seq_len, _p(tree_k), _p(tree_v),
                                        _p(anc_mask), _p(n_nodes), batch, B, Hq, Hkv, D, kv_batch_stride,
                                        softmax_scale, _p(out), _p(lse), _p(device_status), _p(workspace), wb,
                                        _stream(stream), int(flags))
    if check:
        _check(st, "jet_tree_verify_attn_ex")
    return st


def jet_tree_verify_attn_tail_ex(q, k_cache, v_cache, page_table, max_pages_per_seq, page_size, num_pages,
                                 seq_len, max_seq_len, anc_mask, n_nodes, batch, B, Hq, Hkv, D, kv_batch_stride,
                                 softmax_scale, out, lse, device_status, workspace, flags, workspace_bytes=None,
                                 stream=None, check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_verify_attn_tail_ex(_p(q), _p(k_cache), _p(v_cache), _p(page_table), max_pages_per_seq,
                                             page_size, num_pages, _p(seq_len), max_seq_len, _p(anc_mask),
                                             _p(n_nodes), batch, B, Hq, Hkv, D, kv_batch_stride, softmax_scale,
                                             _p(out), _p(lse), _p(device_status), _p(workspace), wb,
                                             _stream(stream), int(flags))
    if check:
        _check(st, "jet_tree_verify_attn_tail_ex")
    return st


def jet_kv_compact_tail(k_cache, v_cache, cache_layer_stride, kv_batch_stride, page_table, max_pages_per_seq,
                        page_size, path, accept_len, seq_len, layers, batch, B, Hkv, D, N, stream=None,
                        check=True):
    st = load().jet_kv_compact_tail(_p(k_cache), _p(v_cache), cache_layer_stride, kv_batch_stride, _p(page_table),
                                    max_pages_per_seq, page_size, _p(path), _p(accept_len), _p(seq_len), layers,
                                    batch, B, Hkv, D, N, _stream(stream))
    if check:
        _check(st, "jet_kv_compact_tail")
    return st


def jet_tree_accept_workspace_bytes(batch, B, V) -> int:
    return load().jet_tree_accept_workspace_bytes(batch, B, V)


def jet_tree_accept(logits, logits_row_stride, token, parent, depth, anc_mask, n_nodes, batch, B, V, N,
                    tgt_argmax, accept_len, path, out_tokens, workspace, workspace_bytes=None, stream=None,
                    check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_accept(_p(logits), logits_row_stride, _p(token), _p(parent), _p(depth), _p(anc_mask),
                                _p(n_nodes), batch, B, V, N, _p(tgt_argmax), _p(accept_len), _p(path),
                                _p(out_tokens), _p(workspace), wb, _stream(stream))
    if check:
        _check(st, "jet_tree_accept")
    return st


def jet_tree_accept_hidden_workspace_bytes(batch, B) -> int:
    return load().jet_tree_accept_hidden_workspace_bytes(batch, B)


def jet_tree_accept_hidden(hidden, lm_head_weight, d, token, parent, depth, anc_mask, n_nodes, batch, B, V, N,
                           tgt_argmax, accept_len, path, out_tokens, device_status, workspace, workspace_bytes=None,
                           stream=None, check=True):
    """Greedy acceptance from the final hidden states: the LM head runs inside the call, only arg-maxima are kept."""
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_accept_hidden(_p(hidden), _p(lm_head_weight), d, _p(token), _p(parent), _p(depth),
                                       _p(anc_mask), _p(n_nodes), batch, B, V, N, _p(tgt_argmax), _p(accept_len),
                                       _p(path), _p(out_tokens), _p(device_status), _p(workspace), wb, _stream(stream))
    if check:
        _check(st, "jet_tree_accept_hidden")
    return st


def jet_tree_accept_static(logits, logits_row_stride, token, parent, depth, anc_mask, n_nodes, batch, B, V, N,
                           tgt_argmax, accept_len, path, out_tokens, stream=None, check=True):
    """jet_tree_accept without a caller workspace: the scratch is an array built into libjet.so.
    For callers that must not allocate device memory (everything already reserved, or no allocator
    calls allowed on the decode loop).  Problems larger than the built-in array give JET_ERR_WORKSPACE;
    calls that overlap on one GPU race on the shared array."""
    st = load().jet_tree_accept_static(_p(logits), logits_row_stride, _p(token), _p(parent), _p(depth),
                                       _p(anc_mask), _p(n_nodes), batch, B, V, N, _p(tgt_argmax),
                                       _p(accept_len), _p(path), _p(out_tokens), _stream(stream))
    if check:
        _check(st, "jet_tree_accept_static")
    return st


def jet_tree_accept_sample_workspace_bytes(batch, B, V) -> int:
    return load().jet_tree_accept_sample_workspace_bytes(batch, B, V)


def jet_tree_accept_sample(logits, logits_row_stride, temperature, draft_logp, logp_batch_stride,
                           logp_depth_stride, token, parent, depth, anc_mask, n_nodes, u_accept, u_sample,
                           batch, B, V, N, alpha, accept_len, path, out_tokens, workspace, workspace_bytes=None,
                           stream=None, check=True):
    wb = workspace_bytes if workspace_bytes is not None else (workspace.numel() * workspace.element_size()
                                                              if workspace is not None else 0)
    st = load().jet_tree_accept_sample(_p(logits), logits_row_stride, temperature, _p(draft_logp),
                                       logp_batch_stride, logp_depth_stride, _p(token), _p(parent), _p(depth),
                                       _p(anc_mask), _p(n_nodes), _p(u_accept), _p(u_sample), batch, B, V, N,
                                       _p(alpha), _p(accept_len), _p(path), _p(out_tokens), _p(workspace), wb,
                                       _stream(stream))
    if check:
        _check(st, "jet_tree_accept_sample")
    return st


def jet_kv_compact(tree_k, tree_v, k_cache, v_cache, cache_layer_stride, kv_batch_stride, page_table,
                   max_pages_per_seq, page_size, path, accept_len, seq_len, layers, batch, B, Hkv, D, N,
                   stream=None, check=True):
    st = load().jet_kv_compact(_p(tree_k), _p(tree_v), _p(k_cache), _p(v_cache), cache_layer_stride,
                               kv_batch_stride, _p(page_table), max_pages_per_seq, page_size, _p(path),
                               _p(accept_len), _p(seq_len), layers, batch, B, Hkv, D, N, _stream(stream))
    if check:
        _check(st, "jet_kv_compact")
    return st
