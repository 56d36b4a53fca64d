"""Oracle: draft-tree construction primitives (TEST INFRASTRUCTURE).

Section 4.1: following EAGLE-2 the draft is a tree built with top-k = 10 expansion, 60 tokens in
total and depth 7. The paper gives no further detail; the reading used: every expanded node
proposes its k most probable next tokens with their log-probabilities; a candidate's score is
the sum of log-probabilities on its root path; after the last level the best-scoring candidates
are kept together with the root (ties: lower candidate index first) and relabelled in
(depth, score descending, candidate index) order, which puts every parent before its children.
"""

from __future__ import annotations

from typing import Tuple

import numpy as np


def topk_logprob(logits: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Row-wise k most probable tokens (ties: lowest token id first) and their log-probabilities
    log softmax(logits) in fp64. logits: float32 [..., V]."""
    x = np.asarray(logits, dtype=np.float32)
    flat = x.reshape(-1, x.shape[-1])
    toks = np.zeros((flat.shape[0], k), dtype=np.int32)
    lps = np.zeros((flat.shape[0], k), dtype=np.float64)
    for r in range(flat.shape[0]):
        row = flat[r].astype(np.float64)
        order = np.argsort(-row, kind="stable")[:k]          # stable: equal values keep index order
        m = row.max()
        lse = m + np.log(np.exp(row - m).sum())
        toks[r] = order
        lps[r] = row[order] - lse
    return toks.reshape(x.shape[:-1] + (k,)), lps.reshape(x.shape[:-1] + (k,))


def rerank_tree(cand_parent, cand_score, cand_token, T: int):
    """Keep the root (candidate 0) and the T-1 best-scoring other candidates, relabel.

    cand_parent[c] < c is the parent candidate of c (cand_parent[0] = -1); cand_score is the
    cumulative log-probability (float32 values compared exactly); returns
    (tree_parent int32 [T], draft_tokens int32 [T], kept candidate ids int32 [T])."""
    cand_parent = [int(x) for x in cand_parent]
    score = np.asarray(cand_score, dtype=np.float32)
    C = len(cand_parent)
    assert C >= T >= 1
    others = sorted(range(1, C), key=lambda c: (-float(score[c]), c))
    kept = [0] + others[: T - 1]
    depth = [0] * C
    for c in range(1, C):
        depth[c] = depth[cand_parent[c]] + 1
    kept.sort(key=lambda c: (depth[c], -float(score[c]), c))
    assert kept[0] == 0
    new_of = {c: i for i, c in enumerate(kept)}
    parent = np.full(T, -1, dtype=np.int32)
    for i, c in enumerate(kept[1:], start=1):
        if cand_parent[c] not in new_of:
            raise ValueError("kept set is not closed under ancestors (scores must not increase along a path)")
        parent[i] = new_of[cand_parent[c]]
    tokens = np.array([int(cand_token[c]) for c in kept], dtype=np.int32)
    return parent, tokens, np.array(kept, dtype=np.int32)
