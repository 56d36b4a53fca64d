"""Helpers shared by the GPU parity tests (input marshalling only)."""

import numpy as np
import torch

import oracle

ATTN_MAX_ABS = 2e-2    # attention tolerance for bf16 inputs / fp32 accumulation / bf16 output
ATTN_MEAN_ABS = 2e-3


def bits_to_torch(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device` (same bytes)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def torch_to_bits(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def mask_to_torch(mask: np.ndarray, device="cuda") -> torch.Tensor:
    """uint64 mask words -> int64 tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(mask).view(np.int64)).to(device)


def oracle_attn_all(q_bits, k_bits, v_bits, prefix_len, masks, scale=None):
    """q_bits [B][H][T][D], k_bits/v_bits [B][H][S][D] (uint16), masks [B][T] -> float64 [B][H][T][D]."""
    B, H, T, D = q_bits.shape
    out = np.zeros((B, H, T, D))
    for b in range(B):
        for h in range(H):
            out[b, h] = oracle.attention.tree_attn_bits(q_bits[b, h], k_bits[b, h], v_bits[b, h],
                                                        int(prefix_len[b]), masks[b], scale)
    return out


def assert_attn_close(got_bits: np.ndarray, ref: np.ndarray, max_abs=ATTN_MAX_ABS, mean_abs=ATTN_MEAN_ABS):
    got = oracle.bf16_bits_to_f64(got_bits)
    assert np.isfinite(got).all(), "non-finite attention output"
    err = np.abs(got - ref)
    assert err.max() <= max_abs, f"max-abs error {err.max():.3e} > {max_abs}"
    assert err.mean() <= mean_abs, f"mean-abs error {err.mean():.3e} > {mean_abs}"
    return float(err.max()), float(err.mean())
