"""GPU: stream order is kept when launches overlap through programmatic dependent launch.

Every trial enqueues, without a host synchronisation in between, the tail of a verify step
(argmax, fused acceptance + compaction), the tree-metadata build of a NEW tree into the same mask
buffer, and then L attention launches in the benchmark's configuration (layer 0 may prefetch
its prefix early, layers 1..L-1 are declared independent of the launch before them and overlap
it). With q = 0, V = 0 on the prefix and V = 1 on the tree slots, node i's output is exactly
(depth_i + 1) / (P + depth_i + 1): it reads back the mask the attention launches saw, with a
margin far above the attention tolerance. Two trees of very different depth alternate, so a
launch that ran before the new mask was written would return the other tree's values.
"""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl

pytestmark = pytest.mark.gpu


def test_mask_written_by_tree_build_is_seen_by_overlapping_attention_launches():
    dev = torch.device("cuda")
    L, B, H, T, D, V, P = 6, 1, 32, 60, 128, 32000, 200
    S_cap = P + 64
    i32 = dict(dtype=torch.int32, device=dev)
    bf = dict(dtype=torch.bfloat16, device=dev)
    trees = [wl.chain_tree(T), wl.star_tree(T)]
    rng = np.random.default_rng(5)
    pars = [torch.tensor(np.asarray(t, dtype=np.int32)[None], **i32) for t in trees]
    want = []
    for t in trees:
        depth = oracle.tree_depth(t).astype(np.float64)
        w = (depth + 1.0) / (P + depth + 1.0)
        want.append(oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(w)))
    assert np.abs(want[0] - want[1]).max() > 0.2
    k = torch.randn((L, B, H, S_cap, D), **bf)
    v = torch.zeros((L, B, H, S_cap, D), **bf)
    v[:, :, :, P:P + T] = 1.0
    q = torch.zeros((L, B, H, T, D), **bf)
    out = torch.zeros_like(q)
    pl = torch.full((B,), P, **i32)
    par = pars[0].clone()
    mask = torch.zeros((B, T), dtype=torch.int64, device=dev)
    status = torch.zeros(1, **i32)
    # tail inputs that accept nothing, so the caches stay as they are
    drafts = torch.tensor(wl.sibling_distinct_tokens(rng, trees[1], V)[None], **i32)
    logits = torch.zeros((B, T, V), device=dev)
    logits[:, :, V - 1] = 5.0
    drafts.clamp_(max=V - 2)
    tok = torch.zeros((B, T), **i32)
    idx = torch.zeros((B, 8), **i32)
    n, nx, nl = torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32)
    desc0 = sv.make_attn_desc(q[0], k[0], v[0], out[0], flags=sv.ATTN_FLAG_PREFIX_STABLE | sv.ATTN_FLAG_HALF_SM)
    desc = sv.make_attn_desc(q[0], k[0], v[0], out[0], flags=sv.ATTN_FLAG_INPUTS_STABLE)
    for trial in range(24):
        which = trial & 1
        out.fill_(-1.0)
        sv.specvlm_argmax(logits, tok)
        sv.specvlm_accept_compact(drafts, par, tok, k, v, pl, idx, n, nx, nl, status)
        par.copy_(pars[which])
        sv.specvlm_tree_build(par, pl, mask, status=status)
        for l in range(L):
            sv.specvlm_tree_verify_attn(q[l], k[l], v[l], pl, par, mask, out[l], status=status,
                                        desc=desc0 if l == 0 else desc)
        torch.cuda.synchronize()
        assert status.item() == 0 and n.item() == 0
        got = out.float().cpu().numpy()[:, 0, :, :, :]          # [L][H][T][D]
        err = np.abs(got - want[which][None, None, :, None]).max(axis=(1, 2, 3))
        assert err.max() < 4e-3, (trial, which, err)


def test_back_to_back_launches_of_mixed_shapes_and_flags():
    """Launches of different shapes, split counts and overlap flags enqueued without a host
    synchronisation in between (each on its own tensors, so every promise the flags make holds):
    whole-SM and half-SM configurations follow one another and overlap; every output must still
    match the oracle."""
    import sys
    import os
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    from util import assert_attn_close, bits_to_torch, mask_to_torch, oracle_attn_all, torch_to_bits
    rng = np.random.default_rng(2024)
    cases = []
    for c in range(18):
        B, H, T = int(rng.integers(1, 4)), int(rng.integers(1, 40)), int(rng.integers(1, 65))
        prefixes = [int(x) for x in rng.integers(0, int(rng.choice([100, 700, 3000])), size=B)]
        S_cap = max(prefixes) + T + int(rng.integers(0, 70))
        parents = [wl.eagle2_like_tree(rng, T, min(6, T - 1)) if T >= 20 else
                   (wl.config1_tree(rng, T, min(4, T - 1)) if T > 1 else wl.single_node_tree()) for _ in range(B)]
        masks = np.array([oracle.tree_mask_bits(p) for p in parents])
        q = wl.normal_bf16_bits(rng, (B, H, T, 128))
        k = wl.normal_bf16_bits(rng, (B, H, S_cap, 128))
        v = wl.normal_bf16_bits(rng, (B, H, S_cap, 128))
        flags = int(rng.choice([0, sv.ATTN_FLAG_PREFIX_STABLE, sv.ATTN_FLAG_INPUTS_STABLE, sv.ATTN_FLAG_INPUTS_STABLE,
                                sv.ATTN_FLAG_PREFIX_STABLE | sv.ATTN_FLAG_HALF_SM]))
        splits = int(rng.choice([0, 0, 1, 2, 4, 8]))
        tq, tk, tv = bits_to_torch(q), bits_to_torch(k), bits_to_torch(v)
        cases.append((q, k, v, prefixes, masks, tq, tk, tv, torch.full_like(tq, 7.0),
                      torch.tensor(prefixes, dtype=torch.int32, device="cuda"), mask_to_torch(masks), flags, splits))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for (_, _, _, _, _, tq, tk, tv, out, tpl, tm, flags, splits) in cases:
        desc = sv.make_attn_desc(tq, tk, tv, out, splits, 0.0, flags)
        sv.specvlm_tree_verify_attn(tq, tk, tv, tpl, None, tm, out, status=status, desc=desc)
    torch.cuda.synchronize()
    assert status.item() == 0
    for (q, k, v, prefixes, masks, _, _, _, out, _, _, _, _) in cases:
        assert_attn_close(torch_to_bits(out), oracle_attn_all(q, k, v, prefixes, masks))
