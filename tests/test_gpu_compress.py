"""GPU parity: parameter-free visual compression (pooling, pruning) against the oracle."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import bits_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,C,ratio", [(576, 4096, 4), (2880, 4096, 20), (2880, 5120, 3), (577, 1024, 5), (7, 8, 1), (5, 16, 9)])
def test_visual_pool_matches_oracle(N, C, ratio):
    rng = np.random.default_rng(N + C + ratio)
    B = 2
    bits = wl.normal_bf16_bits(rng, (B, N, C))
    x = bits_to_torch(bits)
    M = (N + ratio - 1) // ratio
    y = torch.full((B, M, C), 7.0, dtype=torch.bfloat16, device="cuda")
    sv.specvlm_visual_pool(x, ratio, y)
    torch.cuda.synchronize()
    xf = oracle.bf16_bits_to_f64(bits)
    exact = oracle.visual_pool(xf, ratio)
    got_bits = torch_to_bits(y)
    got = oracle.bf16_bits_to_f64(got_bits)
    # fp32 window sums of bf16 values, one multiply by 1/count, one rounding to bf16:
    # half a bf16 ulp of the result plus fp32 rounding relative to the window's mean magnitude
    mag = oracle.visual_pool(np.abs(xf), ratio)
    tol = 2.0 ** -8 * np.abs(exact) * 1.001 + 1e-6 * mag + 1e-30
    assert (np.abs(got - exact) <= tol).all()
    differ = got_bits != oracle.f64_to_bf16_bits(exact)
    assert differ.sum() <= max(2, 2e-3 * differ.size)
    if ratio == 1:
        assert np.array_equal(got_bits, bits)


def test_visual_prune_matches_oracle_and_flags_bad_indices():
    rng = np.random.default_rng(3)
    B, N, C = 3, 2880, 4096
    bits = wl.normal_bf16_bits(rng, (B, N, C))
    x = bits_to_torch(bits)
    for M in (144, 960):                                   # 20x and 3x
        keep = np.stack([np.sort(rng.choice(N, size=M, replace=False)) for _ in range(B)]).astype(np.int32)
        y = torch.zeros((B, M, C), dtype=torch.bfloat16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sv.specvlm_visual_prune(x, torch.from_numpy(keep).cuda(), y, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert np.array_equal(torch_to_bits(y), oracle.visual_prune(bits, keep))
    keep = np.array([[0, N, 5], [1, 2, -1], [3, 4, 5]], dtype=np.int32)
    y = torch.ones((B, 3, C), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_visual_prune(x, torch.from_numpy(keep).cuda(), y, status)
    torch.cuda.synchronize()
    got = torch_to_bits(y)
    assert status.item() != 0 and (got[0, 1] == 0).all() and (got[1, 2] == 0).all()
    assert np.array_equal(got[2], bits[2, 3:6]) and np.array_equal(got[0, 0], bits[0, 0])
