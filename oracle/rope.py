"""Oracle: rotary position embedding at tree positions (TEST INFRASTRUCTURE).

The paper's targets are LLaMA/Vicuna-based LLaVA models (Section 4.1), whose attention
rotates q and k by position before the dot product. The paper does not spell the
rotation out; the reading used: base 10000, head_dim D, "rotate-half" pairing of
element d with element d + D/2, angle = position * base^(-2d/D).
"""

from __future__ import annotations

import numpy as np


def rope_rotate_half(x: np.ndarray, pos: np.ndarray, base: float = 10000.0) -> np.ndarray:
    """x: float64 [..., n, D]; pos: integer [n]. Returns the rotated float64 array."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    d = np.arange(half, dtype=np.float64)
    inv_freq = base ** (-2.0 * d / D)                       # [half]
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]   # [n, half]
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :half], x[..., half:]
    out = np.empty_like(x)
    out[..., :half] = lo * c - hi * s
    out[..., half:] = hi * c + lo * s
    return out
