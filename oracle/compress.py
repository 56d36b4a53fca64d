"""Oracle: parameter-free visual token compression (TEST INFRASTRUCTURE).

Section 3.4 builds the elastic compressor from native operators; the two without parameters are
pruning, which drops tokens at random, and pooling. The paper gives ratios (3x, 5x, 20x) but no
further detail. Reading: pooling is 1-D average pooling along the visual-token axis with window =
stride = ratio, the last window averaging whatever tokens remain; pruning keeps the rows whose
indices are given (the random draw is an input), in the given order.
"""

from __future__ import annotations

import numpy as np


def visual_pool(x: np.ndarray, ratio: int) -> np.ndarray:
    """x: float64 [B][N][C] -> float64 [B][ceil(N / ratio)][C], window means."""
    x = np.asarray(x, dtype=np.float64)
    B, N, C = x.shape
    M = (N + ratio - 1) // ratio
    out = np.zeros((B, M, C))
    for m in range(M):
        out[:, m] = x[:, m * ratio:min((m + 1) * ratio, N)].mean(axis=1)
    return out


def visual_prune(x: np.ndarray, keep_idx: np.ndarray) -> np.ndarray:
    """x: [B][N][C], keep_idx: int [B][M] -> [B][M][C], rows copied bit for bit."""
    x = np.asarray(x)
    return np.stack([x[b][np.asarray(keep_idx[b])] for b in range(x.shape[0])])
