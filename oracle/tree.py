"""Oracle: tree metadata (TEST INFRASTRUCTURE).

The draft is a token tree whose root is the target's most recent token (Section 3.3 (a));
verification uses tree attention (Section 4.1), i.e. each tree token attends to the whole
prefix and, inside the tree, to its ancestors and itself. The paper fixes no data
structure; the reading used here: parent array with parent[0] = -1 and parent[i] < i,
one 64-bit mask word per node (bit t set <=> node t is an ancestor of the node or the
node itself), position of a node = prefix length + its depth.
"""

from __future__ import annotations

import numpy as np


def is_valid_tree(parent) -> bool:
    parent = list(parent)
    if len(parent) == 0 or len(parent) > 64 or parent[0] != -1:
        return False
    return all(0 <= parent[i] < i for i in range(1, len(parent)))


def tree_depth(parent) -> np.ndarray:
    """depth[0] = 0, depth[i] = depth[parent[i]] + 1."""
    T = len(parent)
    depth = np.zeros(T, dtype=np.int32)
    for i in range(1, T):
        depth[i] = depth[parent[i]] + 1
    return depth


def tree_mask_bits(parent) -> np.ndarray:
    """mask[i] has bit t set iff t is i or an ancestor of i (the root included)."""
    T = len(parent)
    mask = np.zeros(T, dtype=np.uint64)
    for i in range(T):
        bits = 0
        t = i
        while t >= 0:
            bits |= 1 << t
            t = int(parent[t])
        mask[i] = np.uint64(bits)
    return mask


def tree_positions(parent, prefix_len: int) -> np.ndarray:
    """Position id of each tree node: prefix length + depth (siblings share a position)."""
    return (int(prefix_len) + tree_depth(parent)).astype(np.int32)
