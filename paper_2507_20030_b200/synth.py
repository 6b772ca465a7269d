"""Seeded synthetic KV-cache inputs shared by the tests, the smoke check and the benchmark.

This module only draws inputs.  It contains none of the method's arithmetic (no
DFT, no update, no reconstruction, no attention, no bin selection), so both the
CUDA path and the CPU oracle can be fed from it without sharing any of their
own code.

The caches imitate two well-known properties of real LLM key caches: a few
large-magnitude channels per head, and rotary position modulation.

* ``V ~ N(0, 1)``.
* ``K0 ~ N(0, 1)``; for every (layer, kv head) four distinct "outlier" channels,
  fixed over tokens and batch, are scaled by 10; then rotary position embedding
  (half-split pairs ``(i, i + d/2)``, ``theta_i = 10000 ** (-2 i / d)``) is
  applied at the absolute token position.
* ``q ~ N(0, 1)``.
* Storage rounding (bf16 round-to-nearest-even) is done once here; the values
  both sides consume are the stored ones.
"""
from __future__ import annotations

import torch

ROPE_BASE = 10000.0
N_OUTLIER = 4
OUTLIER_SCALE = 10.0


def config_seed(config: int, layer: int = 0) -> int:
    """Seed rule used everywhere: 20030*1000 + 100*config + layer."""
    return 20030 * 1000 + 100 * int(config) + int(layer)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def outlier_channels(seed: int, n_kv_heads: int, head_dim: int) -> torch.Tensor:
    """[H, 4] distinct channel indices per head, drawn on the CPU from the seed."""
    g = _gen(seed ^ 0x5EED, "cpu")
    rows = [torch.randperm(head_dim, generator=g)[:N_OUTLIER] for _ in range(n_kv_heads)]
    return torch.stack(rows).to(torch.int64)


def rope_tables(pos0: int, T: int, head_dim: int, device) -> tuple[torch.Tensor, torch.Tensor]:
    """cos/sin of position * theta_i, [T, d/2], computed in float64."""
    half = head_dim // 2
    i = torch.arange(half, dtype=torch.float64, device=device)
    theta = ROPE_BASE ** (-2.0 * i / head_dim)
    pos = torch.arange(pos0, pos0 + T, dtype=torch.float64, device=device)
    ang = pos[:, None] * theta[None, :]
    return torch.cos(ang), torch.sin(ang)


def apply_rope(x: torch.Tensor, pos0: int) -> torch.Tensor:
    """Rotate x [..., T, d] by absolute position pos0 + row index (half-split pairs)."""
    T, d = x.shape[-2], x.shape[-1]
    half = d // 2
    cos, sin = rope_tables(pos0, T, d, x.device)
    cos, sin = cos.to(x.dtype), sin.to(x.dtype)
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * cos - b * sin, b * cos + a * sin], dim=-1)


def make_kv(seed: int, batch: int, n_kv_heads: int, T: int, head_dim: int, *,
            pos0: int = 0, dtype: torch.dtype = torch.float32, device="cpu",
            stream_tag: int = 0) -> tuple[torch.Tensor, torch.Tensor]:
    """K, V of shape [B, H, T, d] in `dtype`, tokens at positions pos0 .. pos0+T-1.

    `stream_tag` separates independent draws that share a seed (e.g. the prefill
    cache and each later decode token)."""
    g = _gen(seed * 1000003 + stream_tag, device)
    shape = (batch, n_kv_heads, T, head_dim)
    k = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    out = outlier_channels(seed, n_kv_heads, head_dim).to(device)
    scale = torch.ones(n_kv_heads, head_dim, device=device, dtype=torch.float32)
    scale.scatter_(1, out, OUTLIER_SCALE)
    k = k * scale[None, :, None, :]
    k = apply_rope(k, pos0)
    return k.to(dtype).contiguous(), v.to(dtype).contiguous()


def make_token(seed: int, step: int, batch: int, n_kv_heads: int, head_dim: int, *,
               pos: int, dtype: torch.dtype = torch.float32, device="cpu"):
    """One decode token's k, v of shape [B, H, d] at absolute position `pos`."""
    k, v = make_kv(seed, batch, n_kv_heads, 1, head_dim, pos0=pos, dtype=dtype,
                   device=device, stream_tag=1 + step)
    return k[:, :, 0, :].contiguous(), v[:, :, 0, :].contiguous()


def make_q(seed: int, step: int, batch: int, n_q_heads: int, head_dim: int, *,
           dtype: torch.dtype = torch.float32, device="cpu") -> torch.Tensor:
    """Query vectors [B, H_q, d] ~ N(0, 1)."""
    g = _gen(seed * 1000003 + 500009 + step, device)
    q = torch.randn((batch, n_q_heads, head_dim), generator=g, device=device, dtype=torch.float32)
    return q.to(dtype).contiguous()
