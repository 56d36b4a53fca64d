"""Seeded input generators: draft trees, draft tokens, target logits, bf16 tensors.

Everything here is input construction. Trees are returned as parent arrays with
parent[0] == -1 and parent[i] < i (node 0 is the root, Section 3.3 (a): the target's first
token is the root of the draft's token tree). No attention, argmax, acceptance or
compaction arithmetic lives in this file.
"""

from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------- bf16 bits


def bf16_bits_from_f32(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (round-to-nearest-even); return uint16 bit patterns.

    NaN inputs are not expected (inputs are synthetic finite values or +-Inf).
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounding = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    return ((u + rounding) >> np.uint64(16)).astype(np.uint16)


def normal_bf16_bits(rng: np.random.Generator, shape: Sequence[int]) -> np.ndarray:
    """N(0,1) samples rounded to bf16, as uint16 bit patterns of the given shape."""
    return bf16_bits_from_f32(rng.standard_normal(size=tuple(shape), dtype=np.float32))


# --------------------------------------------------------------------------- small trees


def single_node_tree() -> np.ndarray:
    return np.array([-1], dtype=np.int32)


def chain_tree(T: int) -> np.ndarray:
    """Node i's parent is i-1: a single root-to-leaf path of T nodes."""
    return np.arange(-1, T - 1, dtype=np.int32)


def star_tree(T: int) -> np.ndarray:
    """Every non-root node is a child of the root."""
    p = np.zeros(T, dtype=np.int32)
    p[0] = -1
    return p


def _relabel(parent: List[int], key: List[Tuple]) -> np.ndarray:
    """Relabel nodes in increasing `key` order (root first); keeps parent < child."""
    order = sorted(range(len(parent)), key=lambda i: key[i])
    assert order[0] == 0
    new_of_old = {old: new for new, old in enumerate(order)}
    out = np.empty(len(parent), dtype=np.int32)
    for old, new in new_of_old.items():
        out[new] = -1 if parent[old] < 0 else new_of_old[parent[old]]
    assert all(out[i] < i for i in range(len(out)))
    return out


def config1_tree(rng: np.random.Generator, T: int = 26, max_depth: int = 5,
                 max_children: int = 4) -> np.ndarray:
    """Random growth tree: a chain to `max_depth` first, then nodes attached to random
    nodes that still have < max_children children and depth < max_depth. Relabelled
    breadth-first so that parent < child."""
    parent = [-1]
    depth = [0]
    nchild = [0]
    for d in range(1, max_depth + 1):
        parent.append(len(parent) - 1)
        depth.append(d)
        nchild.append(0)
        nchild[parent[-1]] += 1
    while len(parent) < T:
        cand = [i for i in range(len(parent)) if nchild[i] < max_children and depth[i] < max_depth]
        p = int(cand[int(rng.integers(len(cand)))])
        parent.append(p)
        depth.append(depth[p] + 1)
        nchild.append(0)
        nchild[p] += 1
    return _relabel(parent, [(depth[i], i) for i in range(len(parent))])


# --------------------------------------------------------------------------- EAGLE-2-like


def eagle2_like_tree(rng: np.random.Generator, T: int = 60, max_depth: int = 6,
                     topk: int = 10) -> np.ndarray:
    """Dynamic draft tree in the style the paper adopts (Section 4.1: top-k 10, 60 tokens).

    Level 1 is `topk` children of the root with random log-probabilities; at each later
    level the `topk` best cumulative-score nodes of the previous level each spawn `topk`
    children; after `max_depth` levels the T-1 best-scoring candidates are kept with the
    root. Cumulative scores strictly decrease from parent to child, so the kept set is
    closed under ancestors. Draws are repeated until the kept tree reaches `max_depth`;
    after 64 failed draws the best depth-`max_depth` chain is forced in.
    """
    for attempt in range(65):
        cand_parent = [-1]
        cand_depth = [0]
        cand_score = [0.0]
        frontier = [0]
        for d in range(1, max_depth + 1):
            new_nodes = []
            for p in frontier:
                lam = rng.uniform(0.5, 1.5)
                raw = -lam * np.arange(topk) + 0.1 * rng.standard_normal(topk)
                logp = raw - np.log(np.sum(np.exp(raw)))          # < 0 for every child
                for r in range(topk):
                    cand_parent.append(p)
                    cand_depth.append(d)
                    cand_score.append(cand_score[p] + float(logp[r]))
                    new_nodes.append(len(cand_parent) - 1)
            new_nodes.sort(key=lambda i: -cand_score[i])
            frontier = new_nodes[:topk]
        ranked = sorted(range(1, len(cand_parent)), key=lambda i: -cand_score[i])
        keep = set(ranked[: T - 1])
        deepest = max(cand_depth[i] for i in keep)
        if deepest < max_depth:
            if attempt < 64:
                continue
            forced = set()
            leaf = max((i for i in range(len(cand_parent)) if cand_depth[i] == max_depth),
                       key=lambda i: cand_score[i])
            while leaf > 0:
                forced.add(leaf)
                leaf = cand_parent[leaf]
            keep |= forced
            while len(keep) > T - 1:
                has_child = {cand_parent[i] for i in keep}
                droppable = [i for i in keep if i not in has_child and i not in forced]
                keep.discard(min(droppable, key=lambda i: cand_score[i]))
        keep_list = [0] + sorted(keep)
        idx_of = {c: k for k, c in enumerate(keep_list)}
        for c in keep_list[1:]:
            assert cand_parent[c] in idx_of, "kept set must be ancestor-closed"
        parent = [-1] + [idx_of[cand_parent[c]] for c in keep_list[1:]]
        key = [(cand_depth[c], -cand_score[c], k) for k, c in enumerate(keep_list)]
        return _relabel(parent, key)
    raise AssertionError("unreachable")


# --------------------------------------------------------------------------- tokens, logits


def _levels(parent: np.ndarray) -> np.ndarray:
    lev = np.zeros(len(parent), dtype=np.int64)
    for i in range(1, len(parent)):
        lev[i] = lev[parent[i]] + 1
    return lev


def sibling_distinct_tokens(rng: np.random.Generator, parent: np.ndarray, V: int) -> np.ndarray:
    """Draft token per node; children of one parent get distinct tokens (they are the
    top-k of one draft distribution). Node 0 carries the root token."""
    T = len(parent)
    tok = np.zeros(T, dtype=np.int32)
    tok[0] = int(rng.integers(V))
    for p in range(T):
        kids = [i for i in range(1, T) if parent[i] == p]
        if kids:
            tok[kids] = rng.choice(V, size=len(kids), replace=False).astype(np.int32)
    return tok


def planted_logits(rng: np.random.Generator, parent: np.ndarray, draft_tokens: np.ndarray,
                   V: int, plant_len: int, bump: float = 8.0
                   ) -> Tuple[np.ndarray, List[int]]:
    """N(0,1) fp32 logits [T][V] with one planted root path of exactly `plant_len` drafts.

    Along a random path to a node at level `plant_len`, the logit of the next path node's
    token is raised by `bump` in the row of the current path node, and then lifted above
    the row's other entries if the bump alone did not win. At the path's last node the
    tokens of all of its children are pushed below the row minimum, so the path cannot
    extend. Returns (logits, planted node list starting at the root).
    """
    T = len(parent)
    lev = _levels(parent)
    logits = rng.standard_normal(size=(T, V), dtype=np.float32)
    at_level = [i for i in range(T) if lev[i] == plant_len]
    if not at_level:
        raise ValueError(f"tree has no node at level {plant_len}")
    node = int(at_level[int(rng.integers(len(at_level)))])
    path = []
    while node >= 0:
        path.append(node)
        node = int(parent[node])
    path.reverse()
    for cur, nxt in zip(path[:-1], path[1:]):
        t = int(draft_tokens[nxt])
        logits[cur, t] += np.float32(bump)
        others = np.delete(logits[cur], t)
        if not logits[cur, t] > others.max():
            logits[cur, t] = others.max() + np.float32(1.0)
    last = path[-1]
    kids = [i for i in range(1, T) if parent[i] == last]
    if kids:
        floor = logits[last].min() - np.float32(1.0)
        logits[last, draft_tokens[kids]] = floor
    return logits, path


# --------------------------------------------------------------------------- prefix lengths


def draw_prefix_lens(cfg, rng: np.random.Generator) -> np.ndarray:
    """Per-sequence prefix lengths P_b for a workload config (int32 [B])."""
    B = cfg.B
    if cfg.prefix_rule == "fixed":
        P = np.full(B, cfg.prefix_nominal)
    elif cfg.prefix_rule == "pm25":
        P = np.rint(cfg.prefix_nominal * rng.uniform(0.75, 1.25, size=B)).astype(np.int64)
    elif cfg.prefix_rule == "cfg4":
        P = 2880 + rng.integers(64, 257, size=B) + rng.integers(0, 201, size=B)
        P[0] = cfg.prefix_nominal
    elif cfg.prefix_rule == "cfg5":
        P = rng.integers(6144, 9729, size=B)
        P[0] = cfg.prefix_nominal
    else:
        raise ValueError(cfg.prefix_rule)
    return P.astype(np.int32)
