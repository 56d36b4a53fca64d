"""Oracle: temperature > 0 tree acceptance by speculative sampling (TEST INFRASTRUCTURE).

Section 3.1 discards incorrect drafted tokens by speculative sampling and Section 4.1 evaluates
stochastic decoding (temperature 1) while preserving the target distribution. The paper gives
no algorithm for trees; the reading used here is the EAGLE-style rule for a tree whose children
are fixed candidates (the top-k of the draft, i.e. proposal probability 1 each): at the current
node with target distribution p = softmax(logits / temperature), the children are tried in index
order; child c with token x is kept with probability p(x) / (1 - mass already rejected); a
rejected token is removed from p. If a child is kept the walk descends to it; otherwise the next
token is drawn from what is left of p (renormalised). The random numbers are inputs: one uniform
per node for its keep/reject test and one uniform per node for the draw made at that node.
Every emitted token is then distributed exactly as the target's own sampling would be.
"""

from __future__ import annotations

from typing import List, Tuple

import numpy as np


def softmax_f64(logits_row, temperature: float) -> np.ndarray:
    z = np.asarray(logits_row, dtype=np.float64) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def accept_sample(parent, draft_tokens, logits, u_accept, u_sample, temperature: float
                  ) -> Tuple[List[int], int, int]:
    """parent, draft_tokens: [T]; logits: [T][V]; u_accept, u_sample: [T] uniforms in [0, 1).
    Returns (kept node path starting at the root, number of kept drafted tokens, next token)."""
    parent = [int(x) for x in parent]
    T = len(parent)
    cur = 0
    path = [0]
    while True:
        p = softmax_f64(logits[cur], temperature)
        removed = 0.0
        gone = set()
        kept = None
        for c in range(1, T):
            if parent[c] != cur:
                continue
            x = int(draft_tokens[c])
            px = 0.0 if x in gone else float(p[x])
            rest = 1.0 - removed
            if rest > 0.0 and float(u_accept[c]) < px / rest:
                kept = c
                break
            removed += px
            gone.add(x)
        if kept is not None:
            path.append(kept)
            cur = kept
            continue
        q = p.copy()
        for x in gone:
            q[x] = 0.0
        target = float(u_sample[cur]) * q.sum()
        cum = np.cumsum(q)
        nxt = int(np.searchsorted(cum, target, side="right"))
        nxt = min(nxt, len(q) - 1)
        while q[nxt] == 0.0 and nxt > 0:       # never return a removed token
            nxt -= 1
        return path, len(path) - 1, nxt


def decision_margins(parent, draft_tokens, logits, u_accept, u_sample, temperature: float) -> float:
    """Smallest distance of any random number used on the walk from its decision boundary
    (relative to the remaining mass). Tests redraw inputs whose margin is too small for a
    float32 implementation to be expected to take the same decisions."""
    parent = [int(x) for x in parent]
    T = len(parent)
    cur, margin = 0, 1.0
    while True:
        p = softmax_f64(logits[cur], temperature)
        removed, gone, kept = 0.0, set(), None
        for c in range(1, T):
            if parent[c] != cur:
                continue
            x = int(draft_tokens[c])
            px = 0.0 if x in gone else float(p[x])
            rest = 1.0 - removed
            thr = px / rest if rest > 0 else 0.0
            margin = min(margin, abs(float(u_accept[c]) - thr))
            if rest > 0.0 and float(u_accept[c]) < thr:
                kept = c
                break
            removed += px
            gone.add(x)
        if kept is not None:
            cur = kept
            continue
        q = p.copy()
        for x in gone:
            q[x] = 0.0
        cum = np.cumsum(q) / q.sum()
        w = float(u_sample[cur])
        margin = min(margin, float(np.abs(cum - w).min()))
        return margin
