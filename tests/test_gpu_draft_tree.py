"""GPU parity: draft-tree construction primitives (top-k log-probabilities, score rerank)."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("V,k,pad", [(32000, 10, 0), (32001, 16, 0), (50, 10, 0), (16, 16, 0), (1000, 1, 0),
                                     (32000, 10, 8), (32000, 7, 3), (40000, 10, 0), (100003, 5, 0),
                                     (151936, 10, 0), (300000, 4, 0)])
def test_topk_logprob_matches_oracle(V, k, pad):
    """Rows of every length class (register-resident shares of 16 to 128 values per thread, and the
    one-block-per-row kernel beyond 262144), aligned and unaligned row strides."""
    rng = np.random.default_rng(V + k)
    rows = 13
    x = (rng.standard_normal((rows, V)) * 2).astype(np.float32)
    x[0, V // 3] = x[0, V // 2] = x[0].max() + 1.0          # equal maxima: lower id first
    x[1, :] = 0.5                                           # constant row: ids 0..k-1
    x[2, V - 1] = 50.0                                      # a dominant last token
    if V >= 1000:
        x[3, 1::2] = -np.inf                                # masked vocabulary entries never win
        x[4, : V - 40] = -np.inf                            # everything finite sits in the last block's share
    if V >= 8192:
        # 16 lanes of one warp own all of the row's largest values (indices 4 t + e + 1024 u for the
        # first block's thread t): too many entries pass the warp's prefilter, so its
        # selection-round path runs
        own = np.array([4 * t + e + 1024 * u for t in range(16) for u in range(4) for e in range(4)])
        x[5, own] += 20.0
        x[6, :64] = 30.0                                    # 64 equal maxima, ids decide
    store = torch.full((rows, V + pad), 1e30, dtype=torch.float32, device="cuda")   # padding must never win
    store[:, :V] = torch.from_numpy(x).cuda()
    lg = store[:, :V]
    toks = torch.full((rows, k), -1, dtype=torch.int32, device="cuda")
    lps = torch.zeros((rows, k), dtype=torch.float32, device="cuda")
    sv.specvlm_topk_logprob(lg, k, toks, lps)
    torch.cuda.synchronize()
    want_t, want_lp = oracle.topk_logprob(x, k)
    assert np.array_equal(toks.cpu().numpy(), want_t)
    assert np.abs(lps.cpu().numpy() - want_lp).max() < 2e-4
    assert toks[1].tolist() == list(range(k))


def _expand(rng, k, levels, V=2000):
    parent, score, token = [-1], [np.float32(0.0)], [int(rng.integers(V))]
    frontier = [0]
    for _ in range(levels):
        new = []
        for p in frontier:
            toks, lps = oracle.topk_logprob(rng.standard_normal(V).astype(np.float32) * 2, k)
            for t, lp in zip(toks, lps):
                parent.append(p); score.append(np.float32(score[p] + lp)); token.append(int(t)); new.append(len(parent) - 1)
        new.sort(key=lambda c: (-float(score[c]), c))
        frontier = new[:k]
    return np.array(parent, dtype=np.int32), np.array(score, dtype=np.float32), np.array(token, dtype=np.int32)


@pytest.mark.parametrize("levels,T", [(6, 60), (7, 61), (2, 8), (6, 64)])
def test_tree_rerank_matches_oracle_bit_exact(levels, T):
    rng = np.random.default_rng(levels * 100 + T)
    B = 6
    cands = [_expand(rng, 10, levels) for _ in range(B)]
    # force exact score ties in one sequence
    cands[1][1][5] = cands[1][1][7]
    C = len(cands[0][0])
    i32 = dict(dtype=torch.int32, device="cuda")
    cp = torch.tensor(np.stack([c[0] for c in cands]), **i32)
    cs = torch.tensor(np.stack([c[1] for c in cands]), dtype=torch.float32, device="cuda")
    ct = torch.tensor(np.stack([c[2] for c in cands]), **i32)
    prefix = rng.integers(0, 9000, size=B).astype(np.int32)
    tp, dt, kept = (torch.full((B, T), -9, **i32) for _ in range(3))
    depth, pos = torch.zeros((B, T), **i32), torch.zeros((B, T), **i32)
    mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
    status = torch.zeros(1, **i32)
    sv.specvlm_tree_rerank(cp, cs, ct, T, tp, dt, kept, mask, depth, pos, torch.tensor(prefix, **i32), status)
    torch.cuda.synchronize()
    assert status.item() == 0 and C == 1 + 10 + 100 * (levels - 1)
    for b in range(B):
        parent, tokens, kept_ids = oracle.rerank_tree(*cands[b], T)
        assert np.array_equal(tp[b].cpu().numpy(), parent)
        assert np.array_equal(dt[b].cpu().numpy(), tokens) and np.array_equal(kept[b].cpu().numpy(), kept_ids)
        assert np.array_equal(mask[b].cpu().numpy().view(np.uint64), oracle.tree_mask_bits(parent))
        assert np.array_equal(depth[b].cpu().numpy(), oracle.tree_depth(parent))
        assert np.array_equal(pos[b].cpu().numpy(), oracle.tree_positions(parent, prefix[b]))
        assert sv.specvlm_tree_validate_host(parent.tolist(), tokens.tolist()) in (0, -4)


def test_tree_rerank_flags_scores_that_increase_along_a_path_and_bad_arguments():
    i32 = dict(dtype=torch.int32, device="cuda")
    cp = torch.tensor([[-1, 0, 1]], **i32)
    cs = torch.tensor([[0.0, -5.0, -1.0]], dtype=torch.float32, device="cuda")
    ct = torch.tensor([[1, 2, 3]], **i32)
    tp, dt = torch.zeros((1, 2), **i32), torch.zeros((1, 2), **i32)
    status = torch.zeros(1, **i32)
    sv.specvlm_tree_rerank(cp, cs, ct, 2, tp, dt, status=status)
    torch.cuda.synchronize()
    assert status.item() & sv.STATUS_BAD_TREE
    with pytest.raises(sv.SpecvlmError):
        sv.specvlm_tree_rerank(cp, cs, ct, 5, tp, dt)           # T > C


@pytest.mark.parametrize("C,T", [(1024, 64), (64, 64), (300, 33), (5, 1), (2, 2)])
def test_tree_rerank_many_exact_ties_and_extreme_sizes(C, T):
    """Scores on a coarse grid (many exactly equal, signed zeros included), so the index part of the
    order decides most of the selection; the candidate limit, C == T and T == 1."""
    rng = np.random.default_rng(C * 100 + T)
    B = 5
    cps, css, cts = [], [], []
    for b in range(B):
        parent = np.full(C, -1, dtype=np.int32)
        score = np.zeros(C, dtype=np.float32)
        for c in range(1, C):
            parent[c] = int(rng.integers(max(0, c - 40), c))
            step = float(rng.integers(0, 3)) * 0.25          # 0 keeps the parent's score exactly
            score[c] = np.float32(score[parent[c]] - step)
        if b == 1:
            score[score == 0] = np.float32(-0.0)             # -0 and +0 compare equal
            score[0] = np.float32(0.0)
        cps.append(parent), css.append(score), cts.append(rng.integers(0, 32000, size=C).astype(np.int32))
    i32 = dict(dtype=torch.int32, device="cuda")
    cp, ct = torch.tensor(np.stack(cps), **i32), torch.tensor(np.stack(cts), **i32)
    cs = torch.tensor(np.stack(css), dtype=torch.float32, device="cuda")
    tp, dt, kept = (torch.full((B, T), -9, **i32) for _ in range(3))
    mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
    status = torch.zeros(1, **i32)
    sv.specvlm_tree_rerank(cp, cs, ct, T, tp, dt, kept, mask, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for b in range(B):
        parent, tokens, kept_ids = oracle.rerank_tree(cps[b], css[b], cts[b], T)
        assert np.array_equal(kept[b].cpu().numpy(), kept_ids)
        assert np.array_equal(tp[b].cpu().numpy(), parent) and np.array_equal(dt[b].cpu().numpy(), tokens)
        assert np.array_equal(mask[b].cpu().numpy().view(np.uint64), oracle.tree_mask_bits(parent))
