"""Device-side buffers of one verify step and the four-call sequence (marshalling only)."""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as clv


def _dev_bf16(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class VerifyStep:
    """Holds the inputs of a workload on one GPU plus every output buffer, and runs
    clv_tree_attn -> clv_accept_argmax -> clv_accept_walk -> clv_kv_commit on the current stream.
    """

    def __init__(self, w, device="cuda", with_lse: bool = True, logits: bool = True):
        c = w.cfg
        self.w = w
        self.device = torch.device(device)
        B, N = c.batch, c.n_nodes
        self.q = _dev_bf16(w.q, device)
        self.k_tree = _dev_bf16(w.k_tree, device)
        self.v_tree = _dev_bf16(w.v_tree, device)
        self.k_cache = _dev_bf16(w.k_cache, device)
        self.v_cache = _dev_bf16(w.v_cache, device)
        self.block_table = (None if w.block_table is None
                            else torch.from_numpy(w.block_table).to(device))
        self.parent = torch.from_numpy(w.parent).to(device)
        self.tokens = torch.from_numpy(w.tokens).to(device)
        self.ctx_len = torch.from_numpy(w.ctx_len).to(device)
        self.logits = _dev_bf16(w.logits, device) if logits else None
        self.ld = w.logits.shape[-1]
        self.max_ctx_len = int(w.ctx_len.max())
        self.scale = float(w.scale)
        self.shape = clv.make_shape(B, N, c.n_q_heads, c.n_kv_heads, c.vocab, w.path_cap)
        self.cache = clv.make_cache(self.k_cache, self.v_cache, self.block_table)
        self.workspace = clv.new_workspace(self.shape, self.cache, self.max_ctx_len, device)
        i32 = dict(dtype=torch.int32, device=device)
        self.out = torch.empty_like(self.q)
        self.lse = torch.empty(B, N, c.n_q_heads, dtype=torch.float32, device=device) if with_lse else None
        self.ids = torch.empty(B, N, **i32)
        self.accept_len = torch.empty(B, **i32)
        self.accept_idx = torch.empty(B, w.path_cap, **i32)
        self.next_token = torch.empty(B, **i32)
        self.ctx_len_out = torch.empty(B, **i32)
        self.status = torch.empty(3, B, **i32)

    def tree_attn(self, stream=None):
        clv.clv_tree_attn(self.shape, self.cache, self.q, self.k_tree, self.v_tree, self.parent,
                          self.ctx_len, self.max_ctx_len, self.scale, self.out, self.lse,
                          self.status[0], self.workspace, stream)

    def accept_argmax(self, stream=None):
        clv.clv_accept_argmax(self.shape, self.logits, self.ld, self.ids, self.workspace, stream)

    def accept_walk(self, stream=None):
        clv.clv_accept_walk(self.shape, self.parent, self.tokens, self.ids, self.accept_len,
                            self.accept_idx, self.next_token, self.status[1], stream)

    def kv_commit(self, stream=None, ctx_len_out: Optional[torch.Tensor] = None):
        clv.clv_kv_commit(self.shape, self.cache, self.k_tree, self.v_tree, self.accept_idx,
                          self.accept_len, self.ctx_len,
                          self.ctx_len_out if ctx_len_out is None else ctx_len_out,
                          self.status[2], stream)

    def accept_walk_commit(self, stream=None, ctx_len_out: Optional[torch.Tensor] = None):
        clv.clv_accept_walk_commit(self.shape, self.cache, self.parent, self.tokens, self.ids, self.k_tree,
                                   self.v_tree, self.ctx_len, self.accept_len, self.accept_idx,
                                   self.next_token, self.ctx_len_out if ctx_len_out is None else ctx_len_out,
                                   self.status[1], self.status[2], stream)

    def run(self, stream=None, fused_tail: bool = True):
        """One whole verify step, stream-ordered: attention, argmax, then the walk and the commit
        (in one launch unless ``fused_tail`` is False)."""
        self.tree_attn(stream)
        self.accept_argmax(stream)
        if fused_tail:
            self.accept_walk_commit(stream)
        else:
            self.accept_walk(stream)
            self.kv_commit(stream)


class ModelVerifyStep:
    """The verify step of a whole model (marshalling only): clv_tree_attn once per layer on that
    layer's Q, tree K/V and cache, the LM head fused with the greedy choice on the nodes' final
    hidden states, the walk, and one commit for the accepted rows of all layers.  The tree may be
    given as depth-first interval labels, which are turned into parent[] on the device first.
    Everything is stream-ordered and can be captured in one CUDA graph.  The layers' other blocks
    (projections, MLP) have no sequence dependency and are not part of this path; the per-layer
    tensors are inputs."""

    def __init__(self, w, layers, hidden_bits, weight_bits, device="cuda", intervals=None):
        q, k_tree, v_tree, k_cache, v_cache = layers
        c = w.cfg
        self.w, self.n_layers = w, q.shape[0]
        B, N = c.batch, c.n_nodes
        self.q, self.k_tree, self.v_tree = (_dev_bf16(x, device) for x in (q, k_tree, v_tree))
        self.k_cache, self.v_cache = _dev_bf16(k_cache, device), _dev_bf16(v_cache, device)
        self.block_table = None if w.block_table is None else torch.from_numpy(w.block_table).to(device)
        self.hidden, self.weight = _dev_bf16(hidden_bits, device), _dev_bf16(weight_bits, device)
        vocab = weight_bits.shape[0]
        i32 = dict(dtype=torch.int32, device=device)
        self.tokens = torch.from_numpy(w.tokens).to(device)
        self.ctx_len = torch.from_numpy(w.ctx_len).to(device)
        self.parent = torch.from_numpy(w.parent).to(device)
        self.tin = self.tout = None
        if intervals is not None:   # the tree arrives as labels; parent[] is derived on the device
            self.tin, self.tout = (torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(device) for x in intervals)
            self.parent = torch.full((B, N), -7, **i32)
        self.max_ctx_len = int(w.ctx_len.max())
        self.scale = float(w.scale)
        self.shape = clv.make_shape(B, N, c.n_q_heads, c.n_kv_heads, vocab, w.path_cap)
        self.caches = [clv.make_cache(self.k_cache[l], self.v_cache[l], self.block_table) for l in range(self.n_layers)]
        self.workspace = clv.new_workspace(self.shape, self.caches[0], self.max_ctx_len, device)
        self.out = torch.empty_like(self.q)
        self.ids = torch.empty(B, N, **i32)
        self.accept_len = torch.empty(B, **i32)
        self.accept_idx = torch.empty(B, w.path_cap, **i32)
        self.next_token = torch.empty(B, **i32)
        self.ctx_len_out = torch.empty(B, **i32)
        self.status = torch.zeros(4 + self.n_layers, B, **i32)   # mask, lm head (word 0 only), walk, commit, attention per layer

    def run(self, stream=None):
        if self.tin is not None:
            clv.clv_tree_from_intervals(self.tin, self.tout, self.parent, self.status[0], stream)
        for l in range(self.n_layers):
            clv.clv_tree_attn(self.shape, self.caches[l], self.q[l], self.k_tree[l], self.v_tree[l], self.parent,
                              self.ctx_len, self.max_ctx_len, self.scale, self.out[l], None,
                              self.status[4 + l], self.workspace, stream)
        clv.clv_lm_head_argmax(self.hidden, self.weight, self.ids.view(-1), self.status[1], self.workspace, stream)
        clv.clv_accept_walk(self.shape, self.parent, self.tokens, self.ids, self.accept_len, self.accept_idx,
                            self.next_token, self.status[2], stream)
        clv.clv_kv_commit_layers(self.shape, self.caches[0], self.n_layers, self.k_cache[0].numel(),
                                 self.k_tree, self.v_tree, self.k_tree[0].numel(), self.accept_idx,
                                 self.accept_len, self.ctx_len, self.ctx_len_out, self.status[3], stream)
