"""Seeded synthetic inputs for the eviction-scoring attention step.

This module only draws random numbers and lays them out; it contains none of the method's
arithmetic (no softmax, no score, no selection), so that the CUDA path and the CPU oracle can both be
fed from it without sharing any code of the method itself.

The shapes follow the attention layers of the models the paper evaluates (Sec. 4.1: Llama-3.1-8B,
Qwen-2.5-7B; budgets 2k-8k; prompt blocks of 128 tokens) and stand in for the paper's long-context
benchmark runs, whose datasets and trained weights are not available here.

Every tensor is drawn with ``torch.randn`` from a ``torch.Generator`` seeded by
``(config seed, stream id, step)``, in fp32, then rounded once to the I/O dtype. The device the
generator lives on changes the bit stream (CPU and CUDA generators differ), so whoever needs the same
data on both sides generates once and copies.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch

# Stream ids: one independent random stream per tensor role.
_S_K0, _S_V0, _S_Q, _S_KNEW, _S_VNEW, _S_MU, _S_LEN, _S_CHAN = range(8)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration (sizes only; see ``WORKLOADS``)."""

    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str  # "bf16" | "f32"
    n_new: int  # m: queries (= new tokens) per step
    budget: int  # tokens kept per (sequence, KV head)
    init_len: int  # tokens already cached before the first step (upper bound when ragged)
    steps: int  # eviction steps in the full workload
    base_mode: str  # "last_query" | "chunk_sum" | "accum" | "external"
    seed: int
    ragged_min_len: Optional[int] = None  # initial lengths uniform in [ragged_min_len, init_len]
    sinks: int = 0  # number of "attention sink" tokens at positions 0..sinks-1
    sink_scale: float = 4.0
    query_shift: float = 2.0
    outlier_channels: int = 0  # key channels scaled by outlier_scale (per KV head)
    outlier_scale: float = 8.0
    layers: int = 1  # independent layers (each with its own seed), processed one after the other

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def capacity(self) -> int:
        # 16-slot granularity keeps every unit's K/V block 16-byte aligned for any dtype
        return ((max(self.init_len, self.budget) + self.n_new + 15) // 16) * 16

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


WORKLOADS: Dict[str, Workload] = {
    # tiny single decode step, fp32; 255 cached + 1 new, evict 128 in one selection
    "c1": Workload("c1", 1, 4, 2, 64, "f32", 1, 128, 255, 1, "last_query", seed=1001),
    # Llama-3-8B-shaped decode at budget 2048 with 4 sink tokens, TOVA-style base score
    "c2": Workload("c2", 1, 32, 8, 128, "bf16", 1, 2048, 2048, 512, "last_query", seed=1002, sinks=4),
    # Llama-3-8B-shaped chunked prefill: 32768-token prompt in blocks of 128, budget 4096, 32 layers
    "c3": Workload("c3", 1, 32, 8, 128, "bf16", 128, 4096, 0, 256, "chunk_sum", seed=1003, layers=32),
    # Qwen2.5-7B-shaped batched decode, ragged lengths, H2O-style accumulated base score
    "c4": Workload("c4", 64, 28, 4, 128, "bf16", 1, 8192, 8192, 256, "accum", seed=1004,
                   ragged_min_len=6144),
    # Llama-3-70B-shaped long-context chunked prefill (131072 tokens, blocks of 512, budget 16384) ...
    "c5p": Workload("c5p", 8, 64, 8, 128, "bf16", 512, 16384, 0, 256, "chunk_sum", seed=1005,
                    outlier_channels=3),
    # ... followed by 1024 decode steps on the full cache
    "c5d": Workload("c5d", 8, 64, 8, 128, "bf16", 1, 16384, 16384, 1024, "last_query", seed=1005,
                    outlier_channels=3),
}


def scaled(w: Workload, **changes) -> Workload:
    """A copy of ``w`` with some sizes replaced (used for reduced parity cases)."""
    return dataclasses.replace(w, **changes)


def _gen(w: Workload, device, stream: int, step: int = 0, layer: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(((w.seed * 64 + layer) * 16 + stream) * 1_000_003 + step)
    return g


def _randn(shape, g: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def mean_query_direction(w: Workload, device, layer: int = 0) -> torch.Tensor:
    """[Hkv, d] unit vectors: the direction the queries of each KV head's group are biased towards."""
    mu = _randn((w.n_kv_heads, w.head_dim), _gen(w, device, _S_MU, 0, layer), device)
    return mu / mu.norm(dim=-1, keepdim=True)


def outlier_channel_mask(w: Workload, device, layer: int = 0) -> torch.Tensor:
    """[Hkv, d] multipliers for the keys: ``outlier_scale`` on ``outlier_channels`` seeded channels."""
    mult = torch.ones((w.n_kv_heads, w.head_dim), device=device, dtype=torch.float32)
    if w.outlier_channels > 0:
        g = _gen(w, device, _S_CHAN, 0, layer)
        for h in range(w.n_kv_heads):
            idx = torch.randperm(w.head_dim, generator=g, device=device)[: w.outlier_channels]
            mult[h, idx] = w.outlier_scale
    return mult


def initial_lengths(w: Workload, device) -> torch.Tensor:
    """[B] int32 cache lengths before the first step."""
    if w.ragged_min_len is None:
        return torch.full((w.batch,), w.init_len, dtype=torch.int32, device=device)
    g = _gen(w, "cpu", _S_LEN)  # lengths are host-side bookkeeping: always the CPU stream
    lens = torch.randint(w.ragged_min_len, w.init_len + 1, (w.batch,), generator=g, dtype=torch.int32)
    return lens.to(device)


def initial_cache(w: Workload, device, layer: int = 0):
    """K, V [B, Hkv, cap, d] (I/O dtype) filled up to ``initial_lengths`` and zero behind."""
    shape = (w.batch, w.n_kv_heads, w.capacity, w.head_dim)
    k = _randn(shape, _gen(w, device, _S_K0, 0, layer), device)
    v = _randn(shape, _gen(w, device, _S_V0, 0, layer), device)
    k = k * outlier_channel_mask(w, device, layer)[None, :, None, :]
    if w.sinks > 0:
        mu = mean_query_direction(w, device, layer)  # [Hkv, d]
        k[:, :, : w.sinks, :] = (w.sink_scale * math.sqrt(w.head_dim)) * mu[None, :, None, :]
    lens = initial_lengths(w, device)
    slot = torch.arange(w.capacity, device=device)[None, None, :, None]
    valid = slot < lens.to(torch.int64)[:, None, None, None]
    k = torch.where(valid, k, torch.zeros_like(k))
    v = torch.where(valid, v, torch.zeros_like(v))
    return k.to(w.torch_dtype).contiguous(), v.to(w.torch_dtype).contiguous()


def step_inputs(w: Workload, device, step: int, layer: int = 0):
    """q [B, Hq, m, d], k_new, v_new [B, Hkv, m, d] (I/O dtype) for eviction step ``step``."""
    m = w.n_new
    q = _randn((w.batch, w.n_q_heads, m, w.head_dim), _gen(w, device, _S_Q, step, layer), device)
    k = _randn((w.batch, w.n_kv_heads, m, w.head_dim), _gen(w, device, _S_KNEW, step, layer), device)
    v = _randn((w.batch, w.n_kv_heads, m, w.head_dim), _gen(w, device, _S_VNEW, step, layer), device)
    k = k * outlier_channel_mask(w, device, layer)[None, :, None, :]
    if w.sinks > 0:
        mu = mean_query_direction(w, device, layer)  # [Hkv, d]
        q = q + w.query_shift * mu.repeat_interleave(w.group, dim=0)[None, :, None, :]
    dt = w.torch_dtype
    return q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous()
