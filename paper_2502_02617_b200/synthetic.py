"""Seeded synthetic inputs shaped like the paper's workloads (Section 5: Llama-3.1-8B style
GQA caches, 8 KV heads x head_dim 128; key caches with a few large-magnitude channels that
the random preconditioning flattens, Fig. 2).

This module only draws random tensors.  It contains none of the method's arithmetic, and it
is the one module that both the CUDA path's callers and the CPU oracle's callers use, so that
both sides see the same bytes.
"""
from __future__ import annotations

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def outlier_channels(seed: int, n_kv_heads: int, d: int, n_outliers: int = 4) -> torch.Tensor:
    """``n_outliers`` distinct channel indices per kv-head (CPU int64 [Hkv, n_outliers])."""
    g = _gen(seed ^ 0x5EED0FF, "cpu")
    n_outliers = min(n_outliers, d)
    return torch.stack([torch.randperm(d, generator=g)[:n_outliers] for _ in range(n_kv_heads)])


def kv_like(seed: int, n_tokens: int, n_kv_heads: int, d: int, dtype=torch.bfloat16,
            device="cpu", n_outliers: int = 4, outlier_scale: float = 10.0):
    """K, V of shape [n_tokens, n_kv_heads, d].  V ~ N(0,1).  K ~ N(0,1) with ``n_outliers``
    channels per head (fixed over tokens) multiplied by ``outlier_scale`` before rounding."""
    g = _gen(seed, device)
    K = torch.randn((n_tokens, n_kv_heads, d), generator=g, device=device, dtype=torch.float32)
    V = torch.randn((n_tokens, n_kv_heads, d), generator=g, device=device, dtype=torch.float32)
    if n_outliers > 0 and outlier_scale != 1.0:
        ch = outlier_channels(seed, n_kv_heads, d, n_outliers).to(device)
        scale = torch.ones((n_kv_heads, d), device=device)
        scale.scatter_(1, ch, outlier_scale)
        K = K * scale[None]
    return K.to(dtype), V.to(dtype)


def queries(seed: int, batch: int, n_q_heads: int, d: int, dtype=torch.bfloat16, device="cpu"):
    """One query token per sequence, N(0,1): [batch, n_q_heads, d]."""
    g = _gen(seed ^ 0xC0FFEE, device)
    return torch.randn((batch, n_q_heads, d), generator=g, device=device,
                       dtype=torch.float32).to(dtype)


def ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> list:
    """Context lengths drawn uniformly from [lo, hi] (inclusive)."""
    g = _gen(seed ^ 0x1E46, "cpu")
    return [int(v) for v in torch.randint(lo, hi + 1, (batch,), generator=g)]
