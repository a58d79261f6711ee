"""Buffer management around the C-ABI calls (allocation and call order only).

A Session owns the device buffers one prompt batch needs and issues the
library calls in path order: score -> search (or apply_lengths) -> compact,
then decode steps.  Nothing here computes on tensors.
"""
from __future__ import annotations

import torch

from . import api


class Session:
    def __init__(self, B, L, H, D, N, dtype, layer_scale, decode_cap, max_budget_rows=None,
                 device="cuda", poison=False, evict_distance=0):
        self.device = torch.device(device)
        self.shape = api.make_shape(B, L, H, D, N, dtype)
        self.B, self.L, self.H, self.D, self.N, self.dtype = B, L, H, D, N, dtype
        dev = self.device
        self.layer_scale = torch.as_tensor(layer_scale, dtype=torch.float32).to(dev).contiguous()
        self.scores = torch.empty((B, L, N), dtype=torch.float32, device=dev)
        self.order = torch.empty((B, L, N), dtype=torch.int32, device=dev)
        self.cum = torch.empty((B, L, N), dtype=torch.int64, device=dev)   # holds uint64 bits
        self.len = torch.empty((B, L), dtype=torch.int32, device=dev)
        self.kept = torch.empty((B, L, N), dtype=torch.int32, device=dev)
        self.p = torch.empty(B, dtype=torch.float64, device=dev)
        self.iters = torch.empty(B, dtype=torch.int32, device=dev)
        self.status = torch.zeros(B, dtype=torch.int32, device=dev)
        self.budget = torch.empty(B, dtype=torch.int64, device=dev)
        self.ws_score = None
        self.ws_compact = api.alloc_workspace(self.shape, api.WS_COMPACT, dev)
        self.ws_decode = api.alloc_workspace(self.shape, api.WS_DECODE, dev)
        rows = L * N if max_budget_rows is None else min(int(max_budget_rows), L * N)
        self.cache = api.alloc_cache(self.shape, B * rows, decode_cap, dev,
                                     fill=float("nan") if poison else None,
                                     evict_distance=evict_distance)
        self.out = torch.empty((B, L, H, D), dtype=dtype, device=dev)

    # -- compress ---------------------------------------------------------
    def score(self, q, k, lse=None):
        if self.ws_score is None:
            self.ws_score = api.alloc_workspace(self.shape, api.WS_SCORE, self.device)
        api.prefixkv_score(self.shape, q, k, self.layer_scale, self.scores, self.ws_score, lse=lse)
        return self.scores

    def search(self, budget_rows, tol=1e-6, max_iters=64, slack_rows=0, scores=None, slack_over_rows=0):
        if isinstance(budget_rows, torch.Tensor):
            self.budget.copy_(budget_rows)
        elif budget_rows is not None:          # None: keep the budget already on the device
            self.budget.fill_(int(budget_rows))
        api.prefixkv_search(self.shape, self.scores if scores is None else scores, self.budget, tol,
                            max_iters, slack_rows, self.order, self.cum, self.len, self.p,
                            self.iters, self.status, slack_over_rows=slack_over_rows)

    def apply_lengths(self, len_in, scores=None):
        len_in = len_in.to(self.device, torch.int32).contiguous()
        api.prefixkv_apply_lengths(self.shape, self.scores if scores is None else scores, len_in,
                                   1 if len_in.dim() == 2 else 0, self.order, self.cum, self.len,
                                   self.status)

    def compact(self, k, v):
        api.prefixkv_compact(self.shape, k, v, self.order, self.len, self.cache, self.status,
                             self.ws_compact, kept=self.kept)

    def compact_merge(self, k, v, mode, match=None):
        api.prefixkv_compact_merge(self.shape, k, v, self.order, self.len, self.cache, mode, self.status,
                                   self.ws_compact, kept=self.kept, match=match)

    def compress(self, q, k, v, budget_rows, tol=1e-6, max_iters=64, slack_rows=0):
        self.score(q, k)
        self.search(budget_rows, tol, max_iters, slack_rows)
        self.compact(k, v)

    # -- decode -----------------------------------------------------------
    def decode(self, q, k_new, v_new, out=None, layer_begin=0, layer_end=None):
        out = self.out if out is None else out
        api.prefixkv_decode_attn(self.shape, self.cache, q, k_new, v_new, self.layer_scale, out,
                                 self.status, self.ws_decode, layer_begin, layer_end)
        return out
