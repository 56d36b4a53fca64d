"""Oracle: temperature-0 acceptance and KV compaction (TEST INFRASTRUCTURE).

Section 3.1 says only that the target verifies the drafted tokens in one pass and that
incorrect tokens are discarded, and the abstract / Section 4.1 that decoding is lossless
with respect to the target. At temperature 0 that fixes the rule: a drafted token is
kept iff it equals the target's greedy choice (argmax of the target logits) at its
parent node, and every one of its ancestors was kept too. The round emits the kept
tokens plus the target's own choice at the last kept node.

Readings where the paper is silent: argmax ties go to the lowest token id; when several
deepest kept nodes exist (possible only if siblings repeat a token) the lowest node
index wins; accept_len counts drafted tokens only (root and bonus token excluded); the
kept nodes' K/V rows move to the slots right after the root's slot, in path order.
"""

from __future__ import annotations

from typing import List, Tuple

import numpy as np


def vocab_argmax(logits: np.ndarray) -> np.ndarray:
    """Row-wise argmax by a sequential scan with strict '>' (first maximum wins;
    -0.0 and +0.0 compare equal). logits: float32 [..., V] without NaN."""
    logits = np.asarray(logits, dtype=np.float32)
    # numpy's argmax returns the first occurrence of the maximum, which is what a
    # sequential scan with strict '>' produces (pinned against such a scan in the tests).
    return np.argmax(logits, axis=-1).astype(np.int32)


def _children(parent, node: int) -> List[int]:
    return [i for i in range(1, len(parent)) if parent[i] == node]


def accept_topdown(parent, draft_tokens, target_tokens) -> Tuple[List[int], int, int]:
    """Walk down from the root through children whose drafted token equals the target's
    greedy token at their parent. Returns (accepted node path starting with the root,
    accept_len = number of drafted tokens kept, next_token = target token at the last
    kept node). If several matching children exist, every one is followed and the
    deepest end node wins (lowest index among equals)."""
    parent = [int(p) for p in parent]

    def descend(node: int, depth: int) -> Tuple[int, int]:
        best = (depth, node)
        for c in _children(parent, node):
            if int(draft_tokens[c]) == int(target_tokens[node]):
                d, n = descend(c, depth + 1)
                if d > best[0] or (d == best[0] and n < best[1]):
                    best = (d, n)
        return best

    depth, node = descend(0, 0)
    path = []
    while node >= 0:
        path.append(node)
        node = parent[node]
    path.reverse()
    return path, depth, int(target_tokens[path[-1]])


def accept_bruteforce(parent, draft_tokens, target_tokens) -> Tuple[List[int], int, int]:
    """Enumerate every root-to-leaf path; on each, count how many leading drafted tokens
    match the target's greedy token at the preceding path node; keep the longest
    (equal lengths: the one whose last matched node has the lowest index)."""
    parent = [int(p) for p in parent]
    T = len(parent)
    leaves = [i for i in range(T) if not _children(parent, i)]
    best_path = [0]
    for leaf in leaves:
        path = []
        n = leaf
        while n >= 0:
            path.append(n)
            n = parent[n]
        path.reverse()
        matched = 0
        for prev, cur in zip(path[:-1], path[1:]):
            if int(draft_tokens[cur]) != int(target_tokens[prev]):
                break
            matched += 1
        cand = path[: matched + 1]
        if len(cand) > len(best_path) or (len(cand) == len(best_path) and cand[-1] < best_path[-1]):
            best_path = cand
    return best_path, len(best_path) - 1, int(target_tokens[best_path[-1]])


def kv_compact(k_cache: np.ndarray, v_cache: np.ndarray, prefix_len, accepted_idx,
               accept_len) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Move the kept nodes' rows next to the root's row.

    k_cache, v_cache: [L][B][H][S_cap][D] (any element dtype; rows are moved bytewise).
    For each sequence b with prefix P_b, and j = 1..accept_len[b], the row in slot
    P_b + accepted_idx[b][j] goes to slot P_b + j. All sources are read before any
    destination is written; every other byte is unchanged. Returns new K, new V and
    new_prefix_len[b] = P_b + 1 + accept_len[b].
    """
    k_new = np.array(k_cache, copy=True)
    v_new = np.array(v_cache, copy=True)
    B = k_cache.shape[1]
    new_len = np.zeros(B, dtype=np.int32)
    for b in range(B):
        P = int(prefix_len[b])
        n = int(accept_len[b])
        saved = []
        for j in range(1, n + 1):
            src = P + int(accepted_idx[b][j])
            saved.append((k_cache[:, b, :, src, :].copy(), v_cache[:, b, :, src, :].copy()))
        for j in range(1, n + 1):
            k_new[:, b, :, P + j, :] = saved[j - 1][0]
            v_new[:, b, :, P + j, :] = saved[j - 1][1]
        new_len[b] = P + 1 + n
    return k_new, v_new, new_len
