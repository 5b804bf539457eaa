"""Oracle, part 4: rotary position embedding of keys and queries.  TEST INFRASTRUCTURE — not a product path.

The paper assigns position ids (Section 6 "Positional Embedding") and leaves the embedding to the base model;
Gemma / LLaMA-style models use the rotate-half form of RoPE, which is what is written out here in float64:

    for i in [0, d/2):   angle = pos * theta ** (-2 i / d)
        y[i]       = x[i] * cos(angle) - x[i + d/2] * sin(angle)
        y[i + d/2] = x[i + d/2] * cos(angle) + x[i] * sin(angle)

The library stores rotated keys as bf16, so `rope_bf16` rounds the float64 result to bf16 (round to nearest even).
"""
from __future__ import annotations

import numpy as np


def rope(x: np.ndarray, pos: np.ndarray, theta: float = 10000.0) -> np.ndarray:
    """x: [n, H, d] float64, pos: [n] integers -> rotated copy, float64."""
    x = np.asarray(x, dtype=np.float64)
    n, _, d = x.shape
    half = d // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]          # [n, d/2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def rope_bf16(x, pos, theta: float = 10000.0):
    """Rotates a torch tensor (any float dtype) in float64 and returns a bf16 torch tensor."""
    import torch
    y = rope(x.detach().to("cpu", torch.float64).numpy(), np.asarray(pos), theta)
    return torch.from_numpy(y).to(torch.bfloat16)
