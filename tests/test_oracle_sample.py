"""Pins for the oracle's temperature > 0 tree acceptance (no GPU needed)."""

import numpy as np
import pytest

import oracle
import workloads as wl


def test_low_temperature_reduces_to_greedy_acceptance():
    rng = np.random.default_rng(1)
    for _ in range(30):
        parent = wl.config1_tree(rng, T=int(rng.integers(4, 20)), max_depth=3)
        draft = wl.sibling_distinct_tokens(rng, parent, 12)
        logits = rng.standard_normal((len(parent), 12)).astype(np.float32) * 3
        greedy = oracle.accept_topdown(parent, draft, oracle.vocab_argmax(logits))
        ua, us = rng.random(len(parent)) * 0.98 + 0.01, rng.random(len(parent)) * 0.98 + 0.01
        got = oracle.accept_sample(parent, draft, logits, ua, us, temperature=1e-3)
        assert got == greedy


def test_single_node_tree_is_inverse_cdf_sampling():
    logits = np.log(np.array([[0.1, 0.2, 0.3, 0.4]]))
    for w, want in [(0.05, 0), (0.15, 1), (0.35, 2), (0.65, 3), (0.999, 3)]:
        path, n, nxt = oracle.accept_sample([-1], [7], logits, [0.5], [w], 1.0)
        assert path == [0] and n == 0 and nxt == want


def test_hand_worked_two_children():
    # root distribution p = (0.5, 0.3, 0.2); children carry tokens 1 and 2 (in that order)
    logits = np.log(np.array([[0.5, 0.3, 0.2]] * 3))
    parent, draft = [-1, 0, 0], [9, 1, 2]
    # u = 0.29 < p(1) = 0.3: child 1 kept; at child 1 (leaf) w = 0.6 -> token 1 (cdf 0.5, 0.8)
    assert oracle.accept_sample(parent, draft, logits, [0, 0.29, 0.0], [0.1, 0.6, 0.1], 1.0) == ([0, 1], 1, 1)
    # u1 = 0.31 rejects token 1; then p(2)/(1-0.3) = 0.2857: u2 = 0.28 keeps child 2
    assert oracle.accept_sample(parent, draft, logits, [0, 0.31, 0.28], [0.1, 0.6, 0.99], 1.0) == ([0, 2], 1, 2)
    # both rejected: what is left is token 0 only
    assert oracle.accept_sample(parent, draft, logits, [0, 0.31, 0.29], [0.7, 0.6, 0.1], 1.0) == ([0], 0, 0)


def test_first_emitted_token_follows_the_target_distribution():
    """Losslessness: whatever the tree, the first token of a round (kept child's token, or the
    token drawn at the root) is distributed as softmax(logits_root / temperature)."""
    rng = np.random.default_rng(2)
    V, n = 6, 60000
    parent = np.array([-1, 0, 0, 0, 1, 1], dtype=np.int32)
    draft = np.array([0, 4, 1, 5, 2, 3], dtype=np.int32)
    logits = rng.standard_normal((6, V)).astype(np.float32)
    for temperature in (1.0, 0.6):
        p = oracle.softmax_f64(logits[0], temperature)
        counts = np.zeros(V)
        second = np.zeros(V)
        n_second = 0
        for _ in range(n):
            path, k, nxt = oracle.accept_sample(parent, draft, logits, rng.random(6), rng.random(6), temperature)
            first = int(draft[path[1]]) if k >= 1 else nxt
            counts[first] += 1
            if k >= 1 and path[1] == 1:            # second token given that child 1 (token 4) was kept
                second[int(draft[path[2]]) if k >= 2 else nxt] += 1
                n_second += 1
        chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
        assert chi2 < 25.0, (temperature, chi2)     # 5 degrees of freedom: P(chi2 > 25) ~ 1e-4
        p1 = oracle.softmax_f64(logits[1], temperature)
        chi2 = ((second - n_second * p1) ** 2 / (n_second * p1)).sum()
        assert chi2 < 25.0, (temperature, chi2)


def test_duplicate_sibling_tokens_and_margins():
    logits = np.log(np.array([[0.5, 0.3, 0.2]] * 3))
    # both children carry token 1: the second try has probability 0
    assert oracle.accept_sample([-1, 0, 0], [9, 1, 1], logits, [0, 0.31, 0.0001], [0.5, 0.5, 0.5], 1.0)[0] == [0]
    m = oracle.decision_margins([-1, 0, 0], [9, 1, 2], logits, [0, 0.29, 0.0], [0.1, 0.6, 0.1], 1.0)
    assert m == pytest.approx(0.01, abs=1e-9)
