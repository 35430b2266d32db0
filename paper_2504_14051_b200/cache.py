"""A budgeted KV cache driven through the C ABI: the call a user of the library makes per step.

Holds the caller-owned device buffers (K, V, base, pos, len, scores, ...) and forwards each step to
``caote_step`` (append the new tokens, score, select, compact), or, for the variants that have no fused entry
point, to the same calls one after the other. No arithmetic happens here.

method: "caote" (Sec. 3.2 score), "fast" (FastCAOTE, Sec. 3.3), "sum_errors" (the per-row errors added up),
"post_evict" (the "caote" step that also returns the attention output over the retained tokens, Sec. 3.1).
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as C


class EvictionCache:
    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, capacity, n_new, dtype, budget,
                 base_mode="last_query", compact_mode="fill", scale: Optional[float] = None,
                 max_evict: Optional[int] = None, device="cuda", method: str = "caote"):
        self.device = torch.device(device)
        scale = head_dim ** -0.5 if scale is None else scale
        self.params = C.make_params(batch, n_q_heads, n_kv_heads, head_dim, capacity, n_new, dtype, scale,
                                    base_mode)
        self.dtype = dtype
        self.compact_mode = C.COMPACT_MODES[compact_mode] if isinstance(compact_mode, str) else compact_mode
        B, Hkv, Hq, d, cap, m = batch, n_kv_heads, n_q_heads, head_dim, capacity, n_new
        dev = self.device
        self.K = torch.zeros((B, Hkv, cap, d), dtype=dtype, device=dev)
        self.V = torch.zeros((B, Hkv, cap, d), dtype=dtype, device=dev)
        self.base = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=dev)
        self.pos = torch.zeros((B, Hkv, cap), dtype=torch.int32, device=dev)
        self.scores = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=dev)
        self.lens = torch.zeros((B,), dtype=torch.int32, device=dev)
        self.n_seen = torch.zeros((B,), dtype=torch.int32, device=dev)
        if isinstance(budget, int):
            budget = torch.full((B,), budget, dtype=torch.int32)
        self.budget = budget.to(device=dev, dtype=torch.int32).contiguous()
        self.max_evict = max_evict if max_evict is not None else max(n_new, 1)
        # what a step hands back (o, evict_idx, n_evict) lives in one buffer, so that a caller who wants it on the
        # host can fetch it with a single copy of `self.results`
        n_o, n_e = B * Hq * m * d, B * Hkv * self.max_evict
        self.results = torch.zeros((n_o + n_e + B,), dtype=torch.float32, device=dev)
        self.o = self.results[:n_o].view(B, Hq, m, d)
        self.evict_idx = self.results[n_o:n_o + n_e].view(torch.int32).view(B, Hkv, self.max_evict)
        self.n_evict = self.results[n_o + n_e:].view(torch.int32)
        self.workspace = C.alloc_workspace(self.params, dev)
        # FastCAOTE (Sec. 3.3) scores against the mean of the cached values: the per-unit sum of V rows is state
        assert method in ("caote", "fast", "sum_errors", "post_evict")
        self.method = method
        self.vsum = torch.zeros((B, Hkv, d), dtype=torch.float32, device=dev) if method == "fast" else None
        self.o_post = torch.zeros_like(self.o) if method == "post_evict" else None

    def load(self, K, V, lens, base=None, pos=None):
        """Install an existing cache state (copied into the owned buffers)."""
        self.K.copy_(K)
        self.V.copy_(V)
        self.lens.copy_(lens)
        self.n_seen.copy_(lens)
        if base is not None:
            self.base.copy_(base)
        if pos is not None:
            self.pos.copy_(pos)
        else:
            cap = self.K.shape[2]
            self.pos.copy_(torch.arange(cap, dtype=torch.int32, device=self.device).expand_as(self.pos))
        if self.vsum is not None:
            C.caote_vsum(self.params, self.V, self.lens, self.vsum)

    def step(self, q, k_new, v_new, stream=None):
        """One eviction step; returns the pre-eviction attention output o [B, Hq, m, d] (method "post_evict":
        the output over the retained tokens)."""
        if self.method in ("sum_errors", "post_evict"):
            p, ws = self.params, self.workspace
            C.caote_append(p, self.K, self.V, self.base, self.pos, self.lens, self.n_seen, k_new, v_new, ws, stream)
            if self.method == "sum_errors":
                C.caote_score_sum_errors(p, q, self.K, self.V, self.lens, self.o, self.scores, ws, stream)
            else:
                C.caote_score(p, q, self.K, self.V, self.lens, self.base, self.o, self.scores, ws, stream)
            C.caote_select_evict(p, self.scores, self.lens, self.budget, self.pos, self.evict_idx, self.n_evict, ws,
                                 stream)
            if self.method == "post_evict":
                C.caote_post_evict_output_ws(p, q, self.K, self.V, self.lens, self.evict_idx, self.n_evict, self.o,
                                             self.o_post, ws, stream)
            C.caote_compact(p, self.K, self.V, self.base, self.pos, self.lens, self.evict_idx, self.n_evict,
                            self.compact_mode, ws, stream)
            return self.o_post if self.method == "post_evict" else self.o
        if self.vsum is not None:
            C.caote_step_fast(self.params, q, k_new, v_new, self.K, self.V, self.base, self.pos, self.lens,
                              self.n_seen, self.budget, self.vsum, self.o, self.scores, self.evict_idx, self.n_evict,
                              self.compact_mode, self.workspace, stream)
            return self.o
        C.caote_step(self.params, q, k_new, v_new, self.K, self.V, self.base, self.pos, self.lens, self.n_seen,
                     self.budget, self.o, self.scores, self.evict_idx, self.n_evict, self.compact_mode,
                     self.workspace, stream)
        return self.o

    def status(self) -> int:
        return C.caote_read_status(self.workspace)
