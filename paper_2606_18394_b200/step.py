"""One verification step = tree_build -> tree_verify_attn per layer -> tree_accept -> kv_compact.

``VerifyStep`` only owns device buffers (torch tensors as memory handles) and issues the four
C-ABI calls in order on the current stream; it performs no arithmetic of its own.  It is what
the benchmark, the smoke check and the end-to-end test drive.
"""
from __future__ import annotations

import math

import torch

from . import binding as jet


class VerifyStep:
    def __init__(self, *, batch, layers, Hq, Hkv, D, B, N, W, V, max_seq_len, page_size=0, num_pages=0,
                 max_pages=0, device="cuda:0", tail=False):
        self.batch, self.layers, self.Hq, self.Hkv, self.D = batch, layers, Hq, Hkv, D
        self.B, self.N, self.W, self.V = B, N, W, V
        self.max_seq_len = max_seq_len
        self.paged = page_size > 0
        # tail: the tree's K/V rows live in the cache behind each prefix (jet_tree_verify_attn_tail /
        # jet_kv_compact_tail); tree_k / tree_v are then only the staging buffers place_tree() copies from
        self.tail = bool(tail)
        self.page_size, self.num_pages, self.max_pages = page_size, num_pages, max_pages
        self.device = torch.device(device)
        dev = self.device
        i32 = dict(dtype=torch.int32, device=dev)
        words = (B + 31) // 32
        self.words = words
        # ---- inputs
        self.logp = torch.zeros((batch, N, V), dtype=torch.float32, device=dev)
        self.root_token = torch.zeros(batch, **i32)
        self.logits = torch.zeros((batch, B, V), dtype=torch.float32, device=dev)
        self.q = torch.zeros((layers, batch, B, Hq, D), dtype=torch.bfloat16, device=dev)
        self.tree_k = torch.zeros((layers, batch, B, Hkv, D), dtype=torch.bfloat16, device=dev)
        self.tree_v = torch.zeros_like(self.tree_k)
        kv_layers = layers
        self.kv_layers = kv_layers
        if self.paged:
            self.k_cache = torch.zeros((kv_layers, num_pages, page_size, Hkv, D), dtype=torch.bfloat16, device=dev)
            self.page_table = torch.zeros((batch, max_pages), **i32)
            self.rows_per_seq = 0
        else:
            # room for the committed path behind the longest prefix
            self.rows_per_seq = max_seq_len + (max(N + 1, B) if self.tail else N + 1)
            self.k_cache = torch.zeros((kv_layers, batch, self.rows_per_seq, Hkv, D), dtype=torch.bfloat16,
                                       device=dev)
            self.page_table = None
        self.v_cache = torch.zeros_like(self.k_cache)
        self.seq_len0 = torch.zeros(batch, **i32)      # prefix lengths at the start of a step
        self.seq_len = torch.zeros(batch, **i32)
        # ---- outputs
        self.parent = torch.zeros((batch, B), **i32)
        self.depth = torch.zeros((batch, B), **i32)
        self.token = torch.zeros((batch, B), **i32)
        self.score = torch.zeros((batch, B), dtype=torch.float32, device=dev)
        self.anc_mask = torch.zeros((batch, B, words), **i32)
        self.n_nodes = torch.zeros(batch, **i32)
        self.out = torch.zeros((layers, batch, B, Hq, D), dtype=torch.bfloat16, device=dev)
        self.status = torch.zeros(1, **i32)
        self.tgt = torch.zeros((batch, B), **i32)
        self.accept_len = torch.zeros(batch, **i32)
        self.path = torch.zeros((batch, N + 1), **i32)
        self.out_tokens = torch.zeros((batch, N + 1), **i32)
        # ---- workspaces
        def ws(nbytes):
            return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=dev)
        self.ws_build = ws(max(jet.jet_tree_build_workspace_bytes(batch, N, V, W),
                               jet.jet_tree_build_scored_workspace_bytes(batch, N, V, W),
                               jet.jet_tree_build_logits_workspace_bytes(batch, N, V, W)))
        # True: `logp` holds the draft head's RAW logits and the tree is built by jet_tree_build_logits
        self.draft_logits = False
        self.depth_lse = torch.zeros((batch, N), dtype=torch.float32, device=dev)
        # expansion score of the tree construction: "accum_logp" (default), "entropy" or "hybrid" (+ score_alpha)
        self.score_mode = "accum_logp"
        self.node_budget = None        # optional i32 [batch]: per-sequence budgets <= B
        self.score_alpha = 0.0
        self.depth_entropy = torch.zeros((batch, N), dtype=torch.float32, device=dev)
        self.ws_attn = ws(jet.jet_tree_verify_attn_workspace_bytes(batch, B, Hq, Hkv, D, self.attn_max_len))
        self.ws_attn.zero_()         # its counters must start at zero; every call leaves them zero
        self.ws_accept = ws(max(jet.jet_tree_accept_workspace_bytes(batch, B, V),
                                jet.jet_tree_accept_sample_workspace_bytes(batch, B, V)))
        # non-greedy acceptance: the caller's random numbers (uniform in [0,1)) and the acceptance ratios
        self.temperature = 1.0
        self.u_accept = torch.zeros((batch, B), dtype=torch.float32, device=dev)
        self.u_sample = torch.zeros((batch,), dtype=torch.float32, device=dev)
        self.alpha = torch.zeros((batch, B), dtype=torch.float32, device=dev)
        self.accept_mode = "greedy"
        # accept_mode "hidden": the acceptance takes the target's final hidden states and applies the LM head itself
        # (enable_lm_head allocates them); no [batch, B, V] logits are needed then
        self.hidden = None
        self.lm_head = None
        self.d_model = 0
        self.ws_accept_hidden = None
        self.scale = 1.0 / math.sqrt(D)
        # Within a step the lengths, the page table and the cached prefix are older than any launch of the
        # layer stack, so every layer but the first (whose predecessor in the stream builds the tree and
        # writes n_nodes) lets the attention kernel read them before its dependency wait.
        self.stable_prefix = True

    @property
    def attn_max_len(self):
        # the bound on the cached keys that the attention call is given: the caller's max_seq_len itself (not
        # the rows a sequence owns, which include room for the commit) -- a call whose bound is exact starts faster
        return self.max_seq_len + (self.B if self.tail else 0)

    def place_tree(self):
        """Tail layout: writes tree_k / tree_v to the cache rows seq_len0[b] + v (what the model's K/V
        projection does in a serving stack; plain torch copies, not part of the timed path's kernels)."""
        assert self.tail
        L = self.seq_len0.to(torch.int64)
        v = torch.arange(self.B, device=self.device, dtype=torch.int64)
        pos = L[:, None] + v[None, :]                                     # [batch, B]
        if self.paged:
            page = torch.gather(self.page_table.to(torch.int64), 1, pos // self.page_size)
            rows = (page * self.page_size + pos % self.page_size).reshape(-1)
            for cache, tree in ((self.k_cache, self.tree_k), (self.v_cache, self.tree_v)):
                flat = cache.view(self.layers, self.num_pages * self.page_size, self.Hkv, self.D)
                flat[:, rows] = tree.reshape(self.layers, -1, self.Hkv, self.D)
        else:
            rows = (torch.arange(self.batch, device=self.device)[:, None] * self.rows_per_seq + pos).reshape(-1)
            for cache, tree in ((self.k_cache, self.tree_k), (self.v_cache, self.tree_v)):
                flat = cache.view(self.layers, self.batch * self.rows_per_seq, self.Hkv, self.D)
                flat[:, rows] = tree.reshape(self.layers, -1, self.Hkv, self.D)

    @property
    def kv_batch_stride(self):
        return 0 if self.paged else self.rows_per_seq * self.Hkv * self.D

    @property
    def cache_layer_stride(self):
        return self.k_cache.stride(0)

    # ------------------------------------------------------------------ the four calls
    def tree_build(self):
        mode = {"accum_logp": 0, "entropy": 1, "hybrid": 2}[self.score_mode]
        if self.draft_logits:
            jet.jet_tree_build_logits(self.logp, self.root_token, self.batch, self.N, self.V, self.W, self.B, mode,
                                      self.score_alpha, self.parent, self.depth, self.token, self.score,
                                      self.anc_mask, self.n_nodes, self.depth_entropy, self.depth_lse,
                                      self.ws_build, node_budget=self.node_budget)
        elif self.score_mode == "accum_logp" and self.node_budget is None:
            jet.jet_tree_build(self.logp, self.root_token, self.batch, self.N, self.V, self.W, self.B, self.parent,
                               self.depth, self.token, self.score, self.anc_mask, self.n_nodes, self.ws_build)
        else:
            jet.jet_tree_build_scored(self.logp, self.root_token, self.batch, self.N, self.V, self.W, self.B, mode,
                                      self.score_alpha, self.parent, self.depth, self.token, self.score,
                                      self.anc_mask, self.n_nodes, self.depth_entropy, self.ws_build,
                                      node_budget=self.node_budget)

    def verify_attn(self, layer, first_in_stack=None):
        """Attention of one layer.  first_in_stack: the launch before this call wrote the tree (default:
        layer == 0), so nothing may be read early."""
        if first_in_stack is None:
            first_in_stack = layer == 0
        flags = jet.JET_ATTN_STABLE_PREFIX if (self.stable_prefix and not first_in_stack) else 0
        if self.tail:
            jet.jet_tree_verify_attn_tail_ex(self.q[layer], self.k_cache[layer], self.v_cache[layer],
                                             self.page_table, self.max_pages, self.page_size, self.num_pages,
                                             self.seq_len, self.attn_max_len, self.anc_mask, self.n_nodes,
                                             self.batch, self.B, self.Hq, self.Hkv, self.D, self.kv_batch_stride,
                                             self.scale, self.out[layer], None, self.status, self.ws_attn, flags)
            return
        jet.jet_tree_verify_attn_ex(self.q[layer], self.k_cache[layer], self.v_cache[layer], self.page_table,
                                    self.max_pages, self.page_size, self.num_pages, self.seq_len,
                                    self.attn_max_len, self.tree_k[layer], self.tree_v[layer], self.anc_mask,
                                    self.n_nodes, self.batch, self.B, self.Hq, self.Hkv, self.D,
                                    self.kv_batch_stride, self.scale, self.out[layer], None, self.status,
                                    self.ws_attn, flags)

    def tree_accept(self):
        jet.jet_tree_accept(self.logits, self.V, self.token, self.parent, self.depth, self.anc_mask, self.n_nodes,
                            self.batch, self.B, self.V, self.N, self.tgt, self.accept_len, self.path,
                            self.out_tokens, self.ws_accept)

    def enable_lm_head(self, d_model):
        """Buffers for accept_mode = "hidden": hidden states [batch * B, d_model] and LM-head weights [V, d_model]."""
        self.d_model = d_model
        self.hidden = torch.zeros((self.batch * self.B, d_model), dtype=torch.bfloat16, device=self.device)
        self.lm_head = torch.zeros((self.V, d_model), dtype=torch.bfloat16, device=self.device)
        self.ws_accept_hidden = torch.empty(max(jet.jet_tree_accept_hidden_workspace_bytes(self.batch, self.B), 256),
                                            dtype=torch.uint8, device=self.device)

    def tree_accept_hidden(self):
        jet.jet_tree_accept_hidden(self.hidden, self.lm_head, self.d_model, self.token, self.parent, self.depth,
                                   self.anc_mask, self.n_nodes, self.batch, self.B, self.V, self.N, self.tgt,
                                   self.accept_len, self.path, self.out_tokens, self.status, self.ws_accept_hidden)

    def tree_accept_sample(self):
        jet.jet_tree_accept_sample(self.logits, self.V, self.temperature, self.logp, self.N * self.V, self.V,
                                   self.token, self.parent, self.depth, self.anc_mask, self.n_nodes, self.u_accept,
                                   self.u_sample, self.batch, self.B, self.V, self.N, self.alpha, self.accept_len,
                                   self.path, self.out_tokens, self.ws_accept)

    def kv_compact(self):
        if self.tail:
            jet.jet_kv_compact_tail(self.k_cache, self.v_cache, self.cache_layer_stride, self.kv_batch_stride,
                                    self.page_table, self.max_pages, self.page_size, self.path, self.accept_len,
                                    self.seq_len, self.layers, self.batch, self.B, self.Hkv, self.D, self.N)
            return
        jet.jet_kv_compact(self.tree_k, self.tree_v, self.k_cache, self.v_cache,
                           self.cache_layer_stride, self.kv_batch_stride,
                           self.page_table, self.max_pages, self.page_size, self.path, self.accept_len,
                           self.seq_len, self.layers, self.batch, self.B, self.Hkv, self.D, self.N)

    def run_front(self):
        """Everything that does not need the target logits: tree construction and the attention of all layers.
        seq_len restarts from seq_len0 so that repeated steps (and graph replays) see the same prefix lengths."""
        self.seq_len.copy_(self.seq_len0)
        self.tree_build()
        for layer in range(self.layers):
            self.verify_attn(layer)

    def run_back(self):
        """Acceptance against the target logits and the commit."""
        if self.accept_mode == "sample":
            self.tree_accept_sample()
        elif self.accept_mode == "hidden":
            self.tree_accept_hidden()
        else:
            self.tree_accept()
        self.kv_compact()

    def run(self):
        """The whole hot path once, on the current stream."""
        self.run_front()
        self.run_back()

    LAUNCHES_PER_STEP_FIXED = 6      # tree_build 2, tree_accept 2, kv_compact 2

    def launches_per_step(self, attn_launches_per_layer=None):
        if attn_launches_per_layer is None:       # what the library says one attention call of this shape enqueues
            attn_launches_per_layer = jet.jet_tree_verify_attn_launches(self.batch, self.B, self.Hq, self.Hkv, self.D,
                                                                        self.attn_max_len)
        return self.LAUNCHES_PER_STEP_FIXED + (1 if self.draft_logits else 0) + self.layers * attn_launches_per_layer
