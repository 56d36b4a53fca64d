"""Pins for the oracle's draft-tree construction primitives (no GPU needed)."""

import itertools

import numpy as np
import pytest
from scipy.special import log_softmax

import oracle


def test_topk_logprob_against_scipy_and_tie_rule():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 4, 500)).astype(np.float32)
    x[0, 0, 17] = x[0, 0, 400] = 9.0                       # equal maxima: lower id first
    toks, lps = oracle.topk_logprob(x, 10)
    assert toks.shape == (3, 4, 10) and toks[0, 0, 0] == 17 and toks[0, 0, 1] == 400
    ref = log_softmax(x.astype(np.float64), axis=-1)
    for idx in itertools.product(range(3), range(4)):
        row = x[idx]
        want = sorted(range(500), key=lambda v: (-float(row[v]), v))[:10]    # plain Python ordering
        assert toks[idx].tolist() == want
        assert np.abs(lps[idx] - ref[idx][want]).max() < 1e-12
        assert (np.diff(lps[idx]) <= 0).all() and np.exp(lps[idx]).sum() <= 1.0


def _expand(rng, k, levels, V=50):
    """Candidate list in EAGLE-2 order: root, its k children, then k children of each of the k
    best nodes of the previous level."""
    parent, score, token = [-1], [np.float32(0.0)], [int(rng.integers(V))]
    frontier = [0]
    for _ in range(levels):
        new = []
        for p in frontier:
            toks, lps = oracle.topk_logprob(rng.standard_normal(V).astype(np.float32), k)
            for t, lp in zip(toks, lps):
                parent.append(p); score.append(np.float32(score[p] + lp)); token.append(int(t)); new.append(len(parent) - 1)
        new.sort(key=lambda c: (-float(score[c]), c))
        frontier = new[:k]
    return np.array(parent), np.array(score, dtype=np.float32), np.array(token)


def test_rerank_gives_a_valid_ancestor_closed_tree_with_the_best_scores():
    rng = np.random.default_rng(2)
    for trial in range(20):
        cp, cs, ct = _expand(rng, k=10, levels=6)
        assert len(cp) == 1 + 10 + 100 * 5
        parent, tokens, kept = oracle.rerank_tree(cp, cs, ct, 60)
        assert oracle.is_valid_tree(parent) and kept[0] == 0 and len(set(kept.tolist())) == 60
        # brute force: the kept set is exactly the 59 largest scores among the candidates
        thresh = np.sort(cs[1:])[::-1][58]
        assert (cs[kept[1:]] >= thresh).all() and (np.delete(cs, kept) <= thresh).all()
        for i in range(1, 60):
            assert kept[parent[i]] == cp[kept[i]] and tokens[i] == ct[kept[i]]
        d = oracle.tree_depth(parent)
        assert (np.diff(d) >= 0).all() and d.max() <= 6


def test_rerank_hand_worked_example():
    #  candidates: 0 root; 1,2 children of 0; 3,4 children of 1; 5 child of 2
    cp = [-1, 0, 0, 1, 1, 2]
    cs = np.array([0.0, -0.2, -1.5, -0.3, -2.0, -1.6], dtype=np.float32)
    ct = [9, 11, 12, 13, 14, 15]
    parent, tokens, kept = oracle.rerank_tree(cp, cs, ct, 4)      # keep 3 best: 1 (-0.2), 3 (-0.3), 2 (-1.5)
    assert kept.tolist() == [0, 1, 2, 3] and parent.tolist() == [-1, 0, 0, 1] and tokens.tolist() == [9, 11, 12, 13]
    parent, tokens, kept = oracle.rerank_tree(cp, cs, ct, 5)      # + candidate 5 (-1.6), child of 2
    assert kept.tolist() == [0, 1, 2, 3, 5] and parent.tolist() == [-1, 0, 0, 1, 2]
    # equal scores: lower candidate index wins the last place
    cs2 = np.array([0.0, -0.2, -1.5, -0.3, -1.5, -1.6], dtype=np.float32)
    assert oracle.rerank_tree(cp, cs2, ct, 4)[2].tolist() == [0, 1, 2, 3]
    with pytest.raises(ValueError):                                 # a child scoring above its parent
        oracle.rerank_tree([-1, 0, 1], np.array([0, -5.0, -1.0], dtype=np.float32), [1, 2, 3], 2)


def test_rerank_chain_and_full_keep():
    cp = [-1, 0, 1, 2, 3]
    cs = -np.arange(5, dtype=np.float32)
    parent, tokens, kept = oracle.rerank_tree(cp, cs, [5, 6, 7, 8, 9], 5)
    assert parent.tolist() == [-1, 0, 1, 2, 3] and kept.tolist() == [0, 1, 2, 3, 4]
