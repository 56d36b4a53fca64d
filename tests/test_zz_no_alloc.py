"""The workspace-free attention entry point against the regular one (GPU).

Some users of the library cannot hand it scratch memory: their own pool already owns the
whole GPU, or they sit in a decode loop where an allocation would stall every stream. For
them `specvlm_tree_verify_attn_static` keeps the split-KV scratch in a fixed array inside
the library. This test calls it through the C ABI twice in a row (the array keeps the
first call's contents, so the second call proves the needed parts are cleared) and compares
each result with the regular entry point's within the attention tolerance of the other
tests. This file is named so that pytest collects it last.
"""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import ATTN_MAX_ABS, ATTN_MEAN_ABS, bits_to_torch, mask_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


def _inputs(seed, B, H, T, prefixes):
    rng = np.random.default_rng(seed)
    S_cap = int(max(prefixes)) + T
    parents = np.array([wl.eagle2_like_tree(rng, T, 6) for _ in range(B)])
    masks = np.array([oracle.tree_mask_bits(p) for p in parents])
    q = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, T, 128)))
    k = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, S_cap, 128)))
    v = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, S_cap, 128)))
    pl = torch.tensor(prefixes, dtype=torch.int32, device="cuda")
    return q, k, v, pl, mask_to_torch(masks)


def _regular(q, k, v, pl, mask, splits):
    out = torch.empty_like(q)
    desc = sv.make_attn_desc(q, k, v, out, splits, 0.0)
    ws = sv.alloc_attn_workspace(desc, q.device)
    sv.specvlm_tree_verify_attn(q, k, v, pl, None, mask, out, workspace=ws, desc=desc)
    torch.cuda.synchronize()
    return oracle.bf16_bits_to_f64(torch_to_bits(out))


def _static(q, k, v, pl, mask, splits):
    out = torch.full_like(q, 3.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_tree_verify_attn_static(q, k, v, pl, None, mask, out, status=status, num_splits=splits)
    torch.cuda.synchronize()
    assert status.item() == 0
    return oracle.bf16_bits_to_f64(torch_to_bits(out))


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    # two different problems back to back: the second one runs on the first one's leftovers
    first = _inputs(101, B=2, H=8, T=60, prefixes=[900, 411])
    second = _inputs(102, B=1, H=16, T=60, prefixes=[1300])
    for case, splits in ((first, 6), (second, 0), (first, 3)):
        want = _regular(*case, splits)
        got = _static(*case, splits)
        err = np.abs(got - want)
        assert np.isfinite(got).all()
        assert err.max() <= ATTN_MAX_ABS and err.mean() <= ATTN_MEAN_ABS
    # and it agrees with the oracle itself on one head
    q, k, v, pl, mask = second
    ref = oracle.attention.tree_attn_bits(torch_to_bits(q)[0, 3], torch_to_bits(k)[0, 3], torch_to_bits(v)[0, 3],
                                          1300, mask.cpu().numpy().view(np.uint64)[0])
    got = _static(*second, 0)[0, 3]
    assert np.abs(got - ref).max() <= ATTN_MAX_ABS and np.abs(got - ref).mean() <= ATTN_MEAN_ABS


def test_static_scratch_entry_point_rejects_oversized_shapes():
    # 16 sequence-heads x 64 splits = 1024 partial slots, twice what the built-in array holds
    q, k, v, pl, mask = _inputs(103, B=2, H=8, T=60, prefixes=[4100, 4100])
    out = torch.empty_like(q)
    with pytest.raises(sv.SpecvlmError, match="exceeds the built-in scratch"):
        sv.specvlm_tree_verify_attn_static(q, k, v, pl, None, mask, out, num_splits=64)
    # the same shape with fewer splits fits and runs
    sv.specvlm_tree_verify_attn_static(q, k, v, pl, None, mask, out, num_splits=8)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
