"""Test-side helpers: run the C-ABI entry points on numpy inputs (device memory via torch)."""
from __future__ import annotations

import numpy as np
import torch

import paper_2606_18394_b200 as jet

DEV = "cuda:0"


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV)


def dev_bf16(bits):
    """uint16 bit patterns -> device bf16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def bf16_to_f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def workspace(nbytes):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=DEV)


# ---------------------------------------------------------------------------------------------------
# Canary margins.  Every output tensor of a call is carved out of a larger buffer whose bytes in front
# of and behind the tensor hold a sentinel; after the call the margins must be untouched.  (An
# out-of-bounds store would otherwise land in the allocator's slack unseen.)
# ---------------------------------------------------------------------------------------------------
_MARGIN = 512            # bytes on either side (keeps the 256-byte alignment of the tensor itself)
_SENTINEL = 0xA5
_guards = []


def guarded_full(shape, fill, dtype):
    """A tensor like torch.full(shape, fill, dtype) on the device, with sentinel margins around it."""
    shape = tuple(int(x) for x in (shape if isinstance(shape, (tuple, list)) else (shape,)))
    item = torch.empty((), dtype=dtype).element_size()
    nbytes = int(np.prod(shape, dtype=np.int64)) * item
    padded = (nbytes + 255) // 256 * 256
    raw = torch.full((_MARGIN + padded + _MARGIN,), _SENTINEL, dtype=torch.uint8, device=DEV)
    body = raw[_MARGIN:_MARGIN + nbytes].view(dtype).view(shape)
    body.fill_(fill)
    _guards.append((raw, nbytes))
    return body


def check_guards():
    """Asserts that no call wrote outside its output tensors; forgets the registered buffers."""
    torch.cuda.synchronize()
    try:
        for raw, nbytes in _guards:
            front = raw[:_MARGIN]
            back = raw[_MARGIN + nbytes:]
            assert bool((front == _SENTINEL).all()), "bytes in front of an output tensor were overwritten"
            assert bool((back == _SENTINEL).all()), "bytes behind an output tensor were overwritten"
    finally:
        _guards.clear()


def run_tree_build(logp, root_token, N, W, B, with_score=True):
    """logp [batch,N,V] fp32 numpy; returns dict of numpy arrays."""
    batch, _, V = logp.shape
    d_logp = dev(logp)
    d_root = dev(np.asarray(root_token, dtype=np.int32))
    words = (B + 31) // 32
    parent = guarded_full((batch, B), -7, torch.int32)
    depth = guarded_full((batch, B), -7, torch.int32)
    token = guarded_full((batch, B), -7, torch.int32)
    score = guarded_full((batch, B), 123.0, torch.float32) if with_score else None
    anc = guarded_full((batch, B, words), 0x5A5A5A5A, torch.int32)
    n_nodes = guarded_full((batch,), -7, torch.int32)
    ws = workspace(jet.jet_tree_build_workspace_bytes(batch, N, V, W))
    jet.jet_tree_build(d_logp, d_root, batch, N, V, W, B, parent, depth, token, score, anc, n_nodes, ws)
    check_guards()
    return dict(parent=parent.cpu().numpy(), depth=depth.cpu().numpy(), token=token.cpu().numpy(),
                score=score.cpu().numpy() if with_score else None,
                anc_mask=anc.cpu().numpy().view(np.uint32), n_nodes=n_nodes.cpu().numpy())


def run_tree_build_scored(logp, root_token, N, W, B, score_mode, alpha, node_budget=None):
    """As run_tree_build, through jet_tree_build_scored; also returns depth_entropy [batch,N]."""
    batch, _, V = logp.shape
    d_logp = dev(logp)
    d_root = dev(np.asarray(root_token, dtype=np.int32))
    words = (B + 31) // 32
    parent = guarded_full((batch, B), -7, torch.int32)
    depth = guarded_full((batch, B), -7, torch.int32)
    token = guarded_full((batch, B), -7, torch.int32)
    score = guarded_full((batch, B), 123.0, torch.float32)
    anc = guarded_full((batch, B, words), 0x5A5A5A5A, torch.int32)
    n_nodes = guarded_full((batch,), -7, torch.int32)
    ent = guarded_full((batch, N), -1.0, torch.float32)
    ws = workspace(jet.jet_tree_build_scored_workspace_bytes(batch, N, V, W))
    jet.jet_tree_build_scored(d_logp, d_root, batch, N, V, W, B, score_mode, alpha, parent, depth, token, score,
                              anc, n_nodes, ent, ws,
                              node_budget=dev(np.asarray(node_budget, dtype=np.int32)) if node_budget is not None else None)
    check_guards()
    return dict(parent=parent.cpu().numpy(), depth=depth.cpu().numpy(), token=token.cpu().numpy(),
                score=score.cpu().numpy(), anc_mask=anc.cpu().numpy().view(np.uint32),
                n_nodes=n_nodes.cpu().numpy(), depth_entropy=ent.cpu().numpy())


def run_tree_build_logits(logits, root_token, N, W, B, score_mode, alpha, node_budget=None):
    """As run_tree_build_scored, through jet_tree_build_logits (raw logits in); also returns depth_lse [batch,N]."""
    batch, _, V = logits.shape
    d_logits = dev(logits)
    d_root = dev(np.asarray(root_token, dtype=np.int32))
    words = (B + 31) // 32
    parent = guarded_full((batch, B), -7, torch.int32)
    depth = guarded_full((batch, B), -7, torch.int32)
    token = guarded_full((batch, B), -7, torch.int32)
    score = guarded_full((batch, B), 123.0, torch.float32)
    anc = guarded_full((batch, B, words), 0x5A5A5A5A, torch.int32)
    n_nodes = guarded_full((batch,), -7, torch.int32)
    ent = guarded_full((batch, N), -1.0, torch.float32)
    lse = guarded_full((batch, N), -1.0, torch.float32)
    ws = workspace(jet.jet_tree_build_logits_workspace_bytes(batch, N, V, W))
    jet.jet_tree_build_logits(d_logits, d_root, batch, N, V, W, B, score_mode, alpha, parent, depth, token, score,
                              anc, n_nodes, ent, lse, ws,
                              node_budget=dev(np.asarray(node_budget, dtype=np.int32)) if node_budget is not None else None)
    check_guards()
    return dict(parent=parent.cpu().numpy(), depth=depth.cpu().numpy(), token=token.cpu().numpy(),
                score=score.cpu().numpy(), anc_mask=anc.cpu().numpy().view(np.uint32),
                n_nodes=n_nodes.cpu().numpy(), depth_entropy=ent.cpu().numpy(), depth_lse=lse.cpu().numpy())


def run_tree_accept(logits, token, parent, depth, anc_mask, n_nodes, N):
    """logits [batch,B,V]; tree arrays [batch,B]; returns dict of numpy arrays."""
    batch, B, V = logits.shape
    d_logits = dev(logits)
    tgt = guarded_full((batch, B), -7, torch.int32)
    acc = guarded_full((batch,), -7, torch.int32)
    path = guarded_full((batch, N + 1), -7, torch.int32)
    toks = guarded_full((batch, N + 1), -7, torch.int32)
    ws = workspace(jet.jet_tree_accept_workspace_bytes(batch, B, V))
    jet.jet_tree_accept(d_logits, V, dev(token.astype(np.int32)), dev(parent.astype(np.int32)),
                        dev(depth.astype(np.int32)), dev(anc_mask.view(np.int32)),
                        dev(np.asarray(n_nodes, dtype=np.int32)), batch, B, V, N, tgt, acc, path, toks, ws)
    check_guards()
    return dict(tgt=tgt.cpu().numpy(), accept_len=acc.cpu().numpy(), path=path.cpu().numpy(),
                out_tokens=toks.cpu().numpy())


def run_tree_accept_sample(logits, temperature, draft_logp, token, parent, depth, anc_mask, n_nodes, N, u_accept,
                           u_sample):
    """logits [batch,B,V], draft_logp [batch,N,V], u_accept [batch,B], u_sample [batch]; returns numpy arrays."""
    batch, B, V = logits.shape
    alpha = guarded_full((batch, B), -7.0, torch.float32)
    acc = guarded_full((batch,), -7, torch.int32)
    path = guarded_full((batch, N + 1), -7, torch.int32)
    toks = guarded_full((batch, N + 1), -7, torch.int32)
    ws = workspace(jet.jet_tree_accept_sample_workspace_bytes(batch, B, V))
    jet.jet_tree_accept_sample(dev(logits), V, float(temperature), dev(draft_logp.astype(np.float32)), N * V, V,
                               dev(token.astype(np.int32)), dev(parent.astype(np.int32)),
                               dev(depth.astype(np.int32)), dev(anc_mask.view(np.int32)),
                               dev(np.asarray(n_nodes, dtype=np.int32)), dev(u_accept.astype(np.float32)),
                               dev(np.asarray(u_sample, dtype=np.float32)), batch, B, V, N, alpha, acc, path,
                               toks, ws)
    check_guards()
    return dict(alpha=alpha.cpu().numpy(), accept_len=acc.cpu().numpy(), path=path.cpu().numpy(),
                out_tokens=toks.cpu().numpy())


def run_kv_compact(tree_k, tree_v, k_cache, v_cache, page_table, path, accept_len, seq_len, N):
    """bf16-bit numpy arrays laid out as the oracle's kv_compact_ref takes them."""
    layers, batch, B, Hkv, D = tree_k.shape
    dk, dv = dev(k_cache.view(np.int16)), dev(v_cache.view(np.int16))
    d_seq = dev(np.asarray(seq_len, dtype=np.int32))
    if page_table is None:
        Lmax = k_cache.shape[2]
        layer_stride = batch * Lmax * Hkv * D
        batch_stride = Lmax * Hkv * D
        pt, max_pages, page_size = None, 0, 0
    else:
        num_pages, page_size = k_cache.shape[1], k_cache.shape[2]
        layer_stride = num_pages * page_size * Hkv * D
        batch_stride = 0
        pt = dev(page_table.astype(np.int32))
        max_pages = page_table.shape[1]
    jet.jet_kv_compact(dev(tree_k.view(np.int16)), dev(tree_v.view(np.int16)), dk, dv, layer_stride,
                       batch_stride, pt, max_pages, page_size, dev(path.astype(np.int32)),
                       dev(np.asarray(accept_len, dtype=np.int32)), d_seq, layers, batch, B, Hkv, D, N)
    check_guards()
    return (dk.cpu().numpy().view(np.uint16), dv.cpu().numpy().view(np.uint16), d_seq.cpu().numpy())


def run_tree_attn(q, k_cache, v_cache, page_table, seq_len, tree_k, tree_v, anc_mask, n_nodes, scale,
                  max_seq_len=None, want_lse=True, flags=0):
    """q [batch,B,Hq,D], tree_k/v [batch,B,Hkv,D] bf16 bits; cache contiguous [batch,Lmax,Hkv,D] or paged
    [num_pages,16,Hkv,D] (with page_table [batch,max_pages]).  Returns (out fp64, lse fp64, status)."""
    batch, B, Hq, D = q.shape
    Hkv = tree_k.shape[2]
    seq_len = np.asarray(seq_len, dtype=np.int32)
    if max_seq_len is None:
        max_seq_len = int(seq_len.max())
    d_q, d_tk, d_tv = dev_bf16(q), dev_bf16(tree_k), dev_bf16(tree_v)
    if k_cache is not None and k_cache.size:
        d_k, d_v = dev_bf16(k_cache), dev_bf16(v_cache)
    else:
        d_k = d_v = None
    if page_table is None:
        pt, max_pages, page_size, num_pages = None, 0, 0, 0
        kv_batch_stride = int(k_cache.shape[1] * Hkv * D) if k_cache is not None else 0
    else:
        pt = dev(page_table.astype(np.int32))
        max_pages, page_size, num_pages = page_table.shape[1], k_cache.shape[1], k_cache.shape[0]
        kv_batch_stride = 0
    out = guarded_full((batch, B, Hq, D), float("nan"), torch.bfloat16)
    lse = guarded_full((batch, Hq, B), float("nan"), torch.float32) if want_lse else None
    status = guarded_full((1,), 0, torch.int32)
    ws = workspace(jet.jet_tree_verify_attn_workspace_bytes(batch, B, Hq, Hkv, D, max_seq_len))
    ws.zero_()          # the attention workspace starts with counters that must be zero
    d_len, d_anc, d_n = dev(seq_len), dev(anc_mask.view(np.int32)), dev(np.asarray(n_nodes, dtype=np.int32))
    torch.cuda.synchronize()      # (with flags: every input is older than the launch before the call)
    if flags:
        jet.jet_tree_verify_attn_ex(d_q, d_k, d_v, pt, max_pages, page_size, num_pages, d_len, max_seq_len,
                                    d_tk, d_tv, d_anc, d_n, batch, B, Hq, Hkv, D, kv_batch_stride, float(scale),
                                    out, lse, status, ws, flags)
    else:
        jet.jet_tree_verify_attn(d_q, d_k, d_v, pt, max_pages, page_size, num_pages, d_len, max_seq_len,
                                 d_tk, d_tv, d_anc, d_n, batch, B, Hq, Hkv, D, kv_batch_stride, float(scale),
                                 out, lse, status, ws)
    check_guards()
    return (bf16_to_f64(out), lse.cpu().numpy().astype(np.float64) if want_lse else None,
            int(status.cpu()[0]))


def run_tree_attn_tail(q, k_cache, v_cache, page_table, seq_len, anc_mask, n_nodes, scale, max_seq_len, Hkv,
                       flags=0):
    """As run_tree_attn for a cache that already holds the tree rows behind each prefix."""
    batch, B, Hq, D = q.shape
    seq_len = np.asarray(seq_len, dtype=np.int32)
    d_q, d_k, d_v = dev_bf16(q), dev_bf16(k_cache), dev_bf16(v_cache)
    if page_table is None:
        pt, max_pages, page_size, num_pages = None, 0, 0, 0
        kv_batch_stride = int(k_cache.shape[1] * Hkv * D)
    else:
        pt = dev(page_table.astype(np.int32))
        max_pages, page_size, num_pages = page_table.shape[1], k_cache.shape[1], k_cache.shape[0]
        kv_batch_stride = 0
    out = guarded_full((batch, B, Hq, D), float("nan"), torch.bfloat16)
    lse = guarded_full((batch, Hq, B), float("nan"), torch.float32)
    status = guarded_full((1,), 0, torch.int32)
    ws = workspace(jet.jet_tree_verify_attn_workspace_bytes(batch, B, Hq, Hkv, D, max_seq_len))
    ws.zero_()
    d_len, d_anc, d_n = dev(seq_len), dev(anc_mask.view(np.int32)), dev(np.asarray(n_nodes, dtype=np.int32))
    torch.cuda.synchronize()
    if flags:
        jet.jet_tree_verify_attn_tail_ex(d_q, d_k, d_v, pt, max_pages, page_size, num_pages, d_len, max_seq_len,
                                         d_anc, d_n, batch, B, Hq, Hkv, D, kv_batch_stride, float(scale), out,
                                         lse, status, ws, flags)
    else:
        jet.jet_tree_verify_attn_tail(d_q, d_k, d_v, pt, max_pages, page_size, num_pages, d_len, max_seq_len,
                                      d_anc, d_n, batch, B, Hq, Hkv, D, kv_batch_stride, float(scale), out,
                                      lse, status, ws)
    check_guards()
    return bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), int(status.cpu()[0])


def run_kv_compact_tail(k_cache, v_cache, page_table, path, accept_len, seq_len, B):
    """k_cache/v_cache [layers, ...] bf16 bits (contiguous [layers,batch,Lmax,Hkv,D] or paged
    [layers,num_pages,page,Hkv,D]); returns new (k, v, seq_len) as numpy."""
    layers = k_cache.shape[0]
    Hkv, D = k_cache.shape[-2], k_cache.shape[-1]
    batch, N = path.shape[0], path.shape[1] - 1
    d_k, d_v = dev(k_cache.view(np.int16)), dev(v_cache.view(np.int16))
    layer_stride = int(np.prod(k_cache.shape[1:]))
    if page_table is None:
        pt, max_pages, page_size = None, 0, 0
        kv_batch_stride = int(np.prod(k_cache.shape[2:]))
    else:
        pt = dev(page_table.astype(np.int32))
        max_pages, page_size = page_table.shape[1], k_cache.shape[2]
        kv_batch_stride = 0
    d_seq = dev(np.asarray(seq_len, dtype=np.int32))
    jet.jet_kv_compact_tail(d_k, d_v, layer_stride, kv_batch_stride, pt, max_pages, page_size,
                            dev(path.astype(np.int32)), dev(np.asarray(accept_len, dtype=np.int32)), d_seq,
                            layers, batch, B, Hkv, D, N)
    check_guards()
    return (d_k.cpu().numpy().view(np.uint16), d_v.cpu().numpy().view(np.uint16), d_seq.cpu().numpy())
