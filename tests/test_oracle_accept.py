"""Pins for the CPU oracle's argmax, acceptance and KV compaction (no GPU needed)."""

import itertools
import os

import numpy as np
import pytest

import oracle
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- argmax


def _scan_argmax(row):
    best = 0
    for j in range(1, len(row)):
        if row[j] > row[best]:
            best = j
    return best


def test_argmax_matches_sequential_scan_and_tie_rules():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 1000), dtype=np.float32)
    x[0, 0, 17] = x[0, 0, 900] = 9.0            # duplicated maximum: first wins
    x[1, 1, 0] = 9.0                            # maximum at index 0
    x[2, 2, 999] = 9.0                          # maximum at the last index
    x[3, 0, :] = -0.0
    x[3, 0, 500] = 0.0                          # -0 == +0: index 0 still wins
    x[4, 1, :] = -np.inf                        # all -inf row -> index 0
    got = oracle.vocab_argmax(x)
    assert got.shape == (5, 3) and got.dtype == np.int32
    for a in range(5):
        for b in range(3):
            assert got[a, b] == _scan_argmax(x[a, b].tolist())
    assert got[0, 0] == 17 and got[1, 1] == 0 and got[2, 2] == 999
    assert got[3, 0] == 0 and got[4, 1] == 0


# ----------------------------------------------------------------------------- acceptance


def test_fully_rejected_tree_gives_zero():
    parent = wl.star_tree(6)
    draft = np.array([5, 10, 11, 12, 13, 14])
    target = np.array([99, 1, 2, 3, 4, 5])       # root's greedy token matches no child
    for f in (oracle.accept_topdown, oracle.accept_bruteforce):
        path, n, nxt = f(parent, draft, target)
        assert path == [0] and n == 0 and nxt == 99


def test_hand_worked_example():
    #        0(t=7)
    #       /      \
    #   1(t=3)     2(t=4)
    #   /    \        \
    # 3(t=8) 4(t=9)   5(t=6)
    parent = [-1, 0, 0, 1, 1, 2]
    draft = [7, 3, 4, 8, 9, 6]
    # target greedy tokens per node: root says 3 (-> node 1), node 1 says 9 (-> node 4),
    # node 4 says 55 (bonus token). Node 2's and 5's rows are irrelevant.
    target = [3, 9, 6, 0, 55, 1]
    for f in (oracle.accept_topdown, oracle.accept_bruteforce):
        assert f(parent, draft, target) == ([0, 1, 4], 2, 55)
    # a match deeper in a rejected branch must not count: root says 4 (-> node 2),
    # node 2 says 5 (no child carries 5) although node 1 -> 4 would have matched
    target = [4, 9, 5, 0, 55, 1]
    for f in (oracle.accept_topdown, oracle.accept_bruteforce):
        assert f(parent, draft, target) == ([0, 2], 1, 5)


def _all_parent_arrays(T):
    for tail in itertools.product(*[range(i) for i in range(1, T)]):
        yield [-1] + list(tail)


def test_bruteforce_equals_topdown_exhaustively_on_tiny_trees():
    rng = np.random.default_rng(2)
    n_checked = 0
    for T in range(1, 7):
        for parent in _all_parent_arrays(T):
            for _ in range(6):
                draft = rng.integers(0, 3, size=T)         # 3 symbols: matches + duplicate siblings
                target = rng.integers(0, 3, size=T)
                a = oracle.accept_topdown(parent, draft, target)
                b = oracle.accept_bruteforce(parent, draft, target)
                assert a == b, (parent, draft, target)
                n_checked += 1
    for parent in itertools.islice(_all_parent_arrays(7), 0, 720, 5):
        draft = rng.integers(0, 3, size=7)
        target = rng.integers(0, 3, size=7)
        assert oracle.accept_topdown(parent, draft, target) == oracle.accept_bruteforce(parent, draft, target)
    assert n_checked > 900


def test_lossless_equals_token_by_token_greedy_decode():
    """The round's output (kept drafts + bonus token) must equal what greedy decoding of
    the target alone emits, where the target's logits for a context are those stored at
    the tree node reached by that context (abstract; Section 4.1: lossless)."""
    rng = np.random.default_rng(3)
    V = 50
    for trial in range(200):
        parent = wl.config1_tree(rng, T=int(rng.integers(6, 27)), max_depth=5)
        draft = wl.sibling_distinct_tokens(rng, parent, 8)   # small vocab: many accidental matches
        logits = rng.standard_normal((len(parent), V)).astype(np.float32)
        logits[:, 8:] -= 10.0                                # greedy tokens fall in the drafted range
        # context (token sequence from the root) -> logits row
        ctx_of = {0: (int(draft[0]),)}
        for i in range(1, len(parent)):
            ctx_of[i] = ctx_of[int(parent[i])] + (int(draft[i]),)
        table = {ctx: logits[i] for i, ctx in ctx_of.items()}
        ctx = (int(draft[0]),)
        emitted = []
        while ctx in table:
            g = int(np.argmax(table[ctx]))
            emitted.append(g)
            ctx = ctx + (g,)
        target = oracle.vocab_argmax(logits)
        path, n, nxt = oracle.accept_topdown(parent, draft, target)
        assert [int(draft[i]) for i in path[1:]] + [nxt] == emitted
        assert n == len(emitted) - 1


@pytest.mark.parametrize("plant_len", [0, 1, 3, 6])
def test_planted_path_is_recovered(plant_len):
    rng = np.random.default_rng(40 + plant_len)
    parent = wl.eagle2_like_tree(rng, T=60, max_depth=6)
    draft = wl.sibling_distinct_tokens(rng, parent, 32000)
    logits, expect = wl.planted_logits(rng, parent, draft, 32000, plant_len)
    target = oracle.vocab_argmax(logits)
    for f in (oracle.accept_topdown, oracle.accept_bruteforce):
        path, n, nxt = f(parent, draft, target)
        assert path == expect and n == plant_len and nxt == int(target[expect[-1]])


def test_mean_accept_len_matches_closed_form():
    """Chain draft with independent per-token match probability alpha: the mean number
    of kept tokens is alpha (1 - alpha^gamma) / (1 - alpha) (Section 3.1, after Eq. 2)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "eq2_sigma.txt")) if l[0] != "#"]
    rng = np.random.default_rng(4)
    for alpha, gamma, sigma in [(float(a), int(g), float(s)) for a, g, s in rows]:
        parent = wl.chain_tree(gamma + 1)
        n_trials = 20000
        total = 0
        sq = 0
        for _ in range(n_trials):
            match = rng.random(gamma) < alpha
            draft = np.arange(100, 100 + gamma + 1)
            target = np.where(np.append(match, False), draft[np.r_[1:gamma + 1, 0]], -1)
            _, n, _ = oracle.accept_topdown(parent, draft, target)
            total += n
            sq += n * n
        mean = total / n_trials
        std = (sq / n_trials - mean * mean) ** 0.5 / n_trials ** 0.5
        assert abs(mean - sigma) < 4.5 * std + 1e-9, (alpha, gamma, mean, sigma)


# ----------------------------------------------------------------------------- compaction


def _slot_tagged_cache(L, B, H, S, D):
    """Every element encodes (layer, b, h, slot, d) so any misplaced row is visible."""
    c = np.zeros((L, B, H, S, D), dtype=np.uint16)
    for l in range(L):
        for b in range(B):
            for h in range(H):
                for s in range(S):
                    c[l, b, h, s, :] = (l * 7919 + b * 1031 + h * 257 + s * 16 + np.arange(D)) % 65521
    return c


def test_compaction_hazard_case_by_hand():
    L, B, H, S, D = 2, 2, 3, 20, 4
    k = _slot_tagged_cache(L, B, H, S, D)
    v = _slot_tagged_cache(L, B, H, S, D) ^ np.uint16(0x5555)
    prefix = np.array([3, 6], dtype=np.int32)
    idx = np.array([[0, 2, 5, 7, -1], [0, 4, -1, -1, -1]], dtype=np.int32)
    n = np.array([3, 1], dtype=np.int32)
    k2, v2, new_len = oracle.kv_compact(k, v, prefix, idx, n)
    assert new_len.tolist() == [7, 8]
    exp_k, exp_v = k.copy(), v.copy()
    for src, dst in [(3 + 2, 3 + 1), (3 + 5, 3 + 2), (3 + 7, 3 + 3)]:   # b = 0, written out by hand
        exp_k[:, 0, :, dst] = k[:, 0, :, src]
        exp_v[:, 0, :, dst] = v[:, 0, :, src]
    exp_k[:, 1, :, 7] = k[:, 1, :, 10]
    exp_v[:, 1, :, 7] = v[:, 1, :, 10]
    assert np.array_equal(k2, exp_k) and np.array_equal(v2, exp_v)
    # slot 3+2 is both a destination (j=2) and a source (j=1): the source was read first
    assert np.array_equal(k2[0, 0, 0, 4], k[0, 0, 0, 5]) and np.array_equal(k2[0, 0, 0, 5], k[0, 0, 0, 8])
    assert np.array_equal(k, _slot_tagged_cache(L, B, H, S, D))        # inputs untouched


def test_compaction_identity_for_fully_accepted_chain_and_zero_accept():
    k = _slot_tagged_cache(1, 1, 2, 16, 4)
    v = k ^ np.uint16(0xFFFF)
    idx = np.array([[0, 1, 2, 3, 4]], dtype=np.int32)
    k2, v2, new_len = oracle.kv_compact(k, v, [5], idx, [4])
    assert np.array_equal(k2, k) and np.array_equal(v2, v) and new_len.tolist() == [10]
    k2, v2, new_len = oracle.kv_compact(k, v, [5], np.array([[0, -1, -1, -1, -1]]), [0])
    assert np.array_equal(k2, k) and np.array_equal(v2, v) and new_len.tolist() == [6]
