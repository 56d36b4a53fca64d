"""Oracle: tree-masked attention over a KV prefix (TEST INFRASTRUCTURE).

What it computes (Section 3.1: the target verifies all drafted tokens in one forward
pass; Section 4.1: tree attention; Section 3.2: attention reads the entire KV cache): for
every tree node i, softmax attention of q_i over the P prefix keys (all visible) and
over the tree keys in cache slots P..P+T-1, of which node i sees slot P+t only if bit t
of its mask word is set. The result has a plain definition, so the oracle is that
definition: the full T x (P+T) score matrix is materialised in fp64, disallowed
entries are set to -inf, a two-pass softmax follows, then the product with V.

bf16 inputs are widened exactly to fp64; nothing is blocked, split or reordered.
"""

from __future__ import annotations

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float64 -> float32 -> bfloat16 (nearest-even at each step); uint16 bits."""
    f = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    return ((u + r) >> np.uint64(16)).astype(np.uint16)


def allowed_matrix(prefix_len: int, mask_bits: np.ndarray, n_keys: int) -> np.ndarray:
    """Boolean [T][n_keys]: key j is visible to node i iff j < P, or j = P + t with
    t < T and bit t of mask_bits[i] set. Keys at or beyond P + T are never visible."""
    T = len(mask_bits)
    P = int(prefix_len)
    allowed = np.zeros((T, n_keys), dtype=bool)
    allowed[:, : min(P, n_keys)] = True
    for i in range(T):
        m = int(mask_bits[i])
        for t in range(T):
            if P + t < n_keys and (m >> t) & 1:
                allowed[i, P + t] = True
    return allowed


def tree_attn(q, k, v, prefix_len: int, mask_bits, scale: float | None = None) -> np.ndarray:
    """One (sequence, head): q float64 [T][D]; k, v float64 [>=P+T][D] (cache slots);
    returns float64 [T][D]. A node with no visible key yields zeros."""
    q = np.asarray(q, dtype=np.float64)
    T, D = q.shape
    P = int(prefix_len)
    n = P + T
    k = np.asarray(k, dtype=np.float64)[:n]
    v = np.asarray(v, dtype=np.float64)[:n]
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    scores = (q @ k.T) * scale                                  # [T][P+T]
    allowed = allowed_matrix(P, mask_bits, n)
    scores = np.where(allowed, scores, -np.inf)
    out = np.zeros((T, D), dtype=np.float64)
    for i in range(T):
        if not allowed[i].any():
            continue
        row = scores[i]
        p = np.exp(row - row.max())                             # exp(-inf) = 0
        p /= p.sum()
        out[i] = p @ v
    return out


def tree_attn_bits(q_bits, k_bits, v_bits, prefix_len: int, mask_bits,
                   scale: float | None = None) -> np.ndarray:
    """Same as tree_attn, from bf16 bit patterns (uint16 arrays)."""
    return tree_attn(bf16_bits_to_f64(q_bits), bf16_bits_to_f64(k_bits),
                     bf16_bits_to_f64(v_bits), prefix_len, mask_bits, scale)


def causal_attn_textbook(q, k, v, scale: float | None = None) -> np.ndarray:
    """Ordinary causal self-attention over one sequence of n tokens, written row by row
    without any mask matrix: token i attends to tokens 0..i. q, k, v float64 [n][D]."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((n, D), dtype=np.float64)
    for i in range(n):
        s = (k[: i + 1] @ q[i]) * scale
        w = np.exp(s - s.max())
        out[i] = (w / w.sum()) @ v[: i + 1]
    return out
