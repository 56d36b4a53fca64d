"""Checks on the seeded input generators (shapes, structure, determinism)."""

import numpy as np

import workloads as wl


def _depths(parent):
    d = [0] * len(parent)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return d


def test_eagle2_like_tree_shape():
    for seed in range(10):
        p = wl.eagle2_like_tree(np.random.default_rng(seed), T=60, max_depth=6, topk=10)
        assert len(p) == 60 and p[0] == -1 and all(0 <= p[i] < i for i in range(1, 60))
        d = _depths(p)
        assert max(d) == 6 and d == sorted(d)
        kids = np.bincount(p[1:], minlength=60)
        assert kids.max() <= 10


def test_config1_tree_shape():
    p = wl.config1_tree(np.random.default_rng(1001), T=26, max_depth=5, max_children=4)
    assert len(p) == 26 and p[0] == -1 and all(0 <= p[i] < i for i in range(1, 26))
    assert max(_depths(p)) == 5 and np.bincount(p[1:]).max() <= 4


def test_generators_are_deterministic():
    a = wl.eagle2_like_tree(np.random.default_rng(5), 60, 6)
    b = wl.eagle2_like_tree(np.random.default_rng(5), 60, 6)
    assert np.array_equal(a, b)
    assert np.array_equal(wl.normal_bf16_bits(np.random.default_rng(9), (4, 8)),
                          wl.normal_bf16_bits(np.random.default_rng(9), (4, 8)))


def test_sibling_tokens_are_distinct():
    rng = np.random.default_rng(2)
    p = wl.eagle2_like_tree(rng, 60, 6)
    tok = wl.sibling_distinct_tokens(rng, p, 12)
    for par in range(60):
        kids = [i for i in range(1, 60) if p[i] == par]
        assert len({int(tok[i]) for i in kids}) == len(kids)


def test_planted_logits_structure():
    rng = np.random.default_rng(3)
    p = wl.eagle2_like_tree(rng, 60, 6)
    tok = wl.sibling_distinct_tokens(rng, p, 32000)
    logits, path = wl.planted_logits(rng, p, tok, 32000, 4)
    assert logits.shape == (60, 32000) and logits.dtype == np.float32
    assert path[0] == 0 and len(path) == 5 and all(p[b] == a for a, b in zip(path[:-1], path[1:]))
    for a, b in zip(path[:-1], path[1:]):
        assert int(np.argmax(logits[a])) == int(tok[b])
    for c in [i for i in range(1, 60) if p[i] == path[-1]]:
        assert logits[path[-1], tok[c]] < logits[path[-1]].max()


def test_prefix_lengths_follow_the_rules():
    rng = np.random.default_rng(0)
    assert wl.draw_prefix_lens(wl.get_config("cfg2"), rng).tolist() == [3008]
    P = wl.draw_prefix_lens(wl.get_config("cfg3_b16_288"), rng)
    assert len(P) == 16 and P.min() >= 312 and P.max() <= 520
    P = wl.draw_prefix_lens(wl.get_config("cfg4"), rng)
    assert P[0] == 3336 and P.min() >= 2944 and P.max() <= 3336
    P = wl.draw_prefix_lens(wl.get_config("cfg5"), rng)
    assert P[0] == 9728 and P.min() >= 6144 and P.max() <= 9728
    for c in wl.CONFIGS.values():
        assert c.s_cap >= int(wl.draw_prefix_lens(c, np.random.default_rng(1)).max()) + c.T


def test_normal_bits_look_standard_normal():
    bits = wl.normal_bf16_bits(np.random.default_rng(4), (200000,))
    f = (bits.astype(np.uint32) << 16).view(np.float32)
    assert abs(float(f.mean())) < 0.01 and abs(float(f.std()) - 1.0) < 0.01
