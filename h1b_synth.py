"""Seeded synthetic inputs for the H1B-KV hot path.

Shapes, value distributions and structure follow the five workload
configurations (7B Llama-2-style decode at 8k context and its relatives);
they stand in for the paper's pretrained checkpoint and text datasets, which
this path does not need.  This module holds no arithmetic of the method: it
only draws random tensors.  Both the CUDA path and the CPU oracle consume what
it returns; neither is imported here.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20251005


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    sketch_bits: int
    group_size: int
    batch: int
    context: int                 # cached tokens per sequence (maximum for ragged batches)
    context_min: int = 0         # > 0: ragged lengths uniform in [context_min, context]
    outlier_frac: float = 0.0    # fraction of (head, channel) positions scaled by outlier_scale
    outlier_scale: float = 8.0
    decode_steps: int = 1
    index: int = 0
    notes: str = field(default="", compare=False)


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", 1, 1, 1, 128, 128, 32, 1, 512, index=1,
                        notes="single head, 512 tokens, one decode step"),
    "c2_7b_8k": Workload("c2_7b_8k", 32, 32, 32, 128, 128, 32, 1, 8192, outlier_frac=0.01, index=2,
                         notes="7B shape, batch 1, 8k context, 1% outlier channels x8"),
    "c3_7b_batched": Workload("c3_7b_batched", 32, 32, 32, 128, 128, 32, 16, 8192, context_min=4096,
                              decode_steps=64, index=3, notes="batch 16, ragged 4096..8192, 64 steps"),
    "c4_gqa_32k": Workload("c4_gqa_32k", 32, 32, 8, 128, 256, 32, 8, 32768, index=4,
                           notes="GQA 32/8, m=256, 32k context, batch 8"),
    "c5_prefill": Workload("c5_prefill", 32, 32, 32, 128, 128, 32, 1, 8192, index=5,
                           notes="prefill compression of 8192 tokens per layer, then one decode"),
    # the paper's small model (12 layers, 8 heads of dimension 64, sketch width 256, 8k context); a batch of 32
    # sequences, so that the cache (1.8 GB) does not sit in the L2
    "c6_60m_8k": Workload("c6_60m_8k", 12, 8, 8, 64, 256, 32, 32, 8192, index=6,
                          notes="60M GPT-2-style shape, head dimension 64, m=256, 8k context, batch 32"),
}


def layer_seed(w: Workload, layer: int, stream: int = 0) -> int:
    """One seed per (workload, layer, stream)."""
    return BASE_SEED + 1000 * w.index + layer + 100003 * stream


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def projection(seed: int, d: int, m: int) -> np.ndarray:
    """The fixed Gaussian matrix, N(0,1), as float32 [d, m] (row i = input channel)."""
    g = _gen(seed, "cpu")
    return torch.randn((d, m), generator=g, dtype=torch.float32).numpy().copy()


def outlier_mask(seed: int, n_heads: int, d: int, frac: float) -> torch.Tensor:
    """Boolean [n_heads, d]: round(frac * n_heads * d) seeded positions."""
    n = n_heads * d
    k = int(round(frac * n))
    mask = torch.zeros(n, dtype=torch.bool)
    if k > 0:
        g = _gen(seed, "cpu")
        mask[torch.randperm(n, generator=g)[:k]] = True
    return mask.view(n_heads, d)


def normal_fp16(seed: int, shape, device: str = "cpu") -> torch.Tensor:
    """N(0,1) drawn in float32 from a seeded generator, rounded to fp16."""
    g = _gen(seed, device)
    return torch.randn(tuple(shape), generator=g, dtype=torch.float32, device=device).to(torch.float16)


def kv_rows(w: Workload, layer: int, n_tokens: int, device: str = "cpu", stream: int = 0,
            batch: int | None = None):
    """K, V as fp16 [B, n_tokens, Hkv, d] for one layer (outlier channels applied)."""
    B = w.batch if batch is None else batch
    shape = (B, n_tokens, w.n_kv_heads, w.head_dim)
    K = normal_fp16(layer_seed(w, layer, 2 * stream + 1), shape, device)
    V = normal_fp16(layer_seed(w, layer, 2 * stream + 2), shape, device)
    if w.outlier_frac > 0:
        mask = outlier_mask(layer_seed(w, layer, 9001), w.n_kv_heads, w.head_dim, w.outlier_frac)
        scale = torch.ones(w.n_kv_heads, w.head_dim, dtype=torch.float16)
        scale[mask] = w.outlier_scale
        scale = scale.to(device)
        K = K * scale                       # fp16 times a power of two: exact
        V = V * scale
    return K.contiguous(), V.contiguous()


def queries(w: Workload, layer: int, device: str = "cpu", stream: int = 0, batch: int | None = None):
    """q as fp16 [B, Hq, d] for one layer."""
    B = w.batch if batch is None else batch
    return normal_fp16(layer_seed(w, layer, 7001 + stream), (B, w.n_q_heads, w.head_dim), device)


def rope_table(n_positions: int, half: int, base: float = 10000.0) -> np.ndarray:
    """Input data for the rotary-embedding option: fp32 [n_positions, half, 2], (cos, sin) of the angle
    position * base^(-i / half) of pair i (the usual geometric frequencies), evaluated in fp64 and rounded once."""
    ang = np.arange(n_positions, dtype=np.float64)[:, None] * base ** (-np.arange(half, dtype=np.float64) / half)[None, :]
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)


def lengths(w: Workload, batch: int | None = None) -> np.ndarray:
    """Cached tokens per sequence: constant, or uniform in [context_min, context]."""
    B = w.batch if batch is None else batch
    if w.context_min <= 0:
        return np.full((B,), w.context, dtype=np.int32)
    g = _gen(BASE_SEED + 1000 * w.index + 777, "cpu")
    r = torch.randint(w.context_min, w.context + 1, (B,), generator=g)
    return r.numpy().astype(np.int32)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller cases for tests)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)
