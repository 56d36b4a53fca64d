"""Pins for the CPU oracle's tree metadata, RoPE and attention (no GPU needed).

Each test checks the oracle against something other than its own formula: a separately
written textbook routine, pure-Python brute force, closed forms, invariances, or
hand-derived fixtures.
"""

import math
import os

import numpy as np
import pytest

import oracle
from oracle.attention import tree_attn_bits
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_f64_from_bf16(rng, shape):
    return oracle.bf16_bits_to_f64(wl.normal_bf16_bits(rng, shape))


# ----------------------------------------------------------------------------- metadata


def test_tree_metadata_matches_hand_derived_fixture():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "tree_example.txt")) if l[0] != "#"]
    parent = [int(r[1]) for r in rows]
    assert oracle.is_valid_tree(parent)
    assert list(oracle.tree_depth(parent)) == [int(r[2]) for r in rows]
    assert [int(m) for m in oracle.tree_mask_bits(parent)] == [int(r[3]) for r in rows]
    assert list(oracle.tree_positions(parent, 100)) == [100 + int(r[2]) for r in rows]


def test_mask_special_shapes():
    T = 9
    chain = oracle.tree_mask_bits(wl.chain_tree(T))
    assert [int(m) for m in chain] == [(1 << (i + 1)) - 1 for i in range(T)]
    star = oracle.tree_mask_bits(wl.star_tree(T))
    assert [int(m) for m in star] == [1] + [1 | (1 << i) for i in range(1, T)]
    # 64-node chain uses the top bit without overflow
    m64 = oracle.tree_mask_bits(wl.chain_tree(64))
    assert int(m64[63]) == (1 << 64) - 1


def test_mask_popcount_is_depth_plus_one_on_random_trees():
    rng = np.random.default_rng(7)
    for _ in range(20):
        parent = wl.eagle2_like_tree(rng, T=60, max_depth=6)
        depth = oracle.tree_depth(parent)
        mask = oracle.tree_mask_bits(parent)
        assert depth.max() == 6
        for i in range(60):
            assert bin(int(mask[i])).count("1") == depth[i] + 1
            assert (int(mask[i]) >> i) & 1 and int(mask[i]) & 1
            if i:
                assert int(mask[i]) == int(mask[parent[i]]) | (1 << i)


def test_invalid_trees_rejected():
    assert not oracle.is_valid_tree([0, 0])
    assert not oracle.is_valid_tree([-1, 1])
    assert not oracle.is_valid_tree([-1, 2, 1])
    assert not oracle.is_valid_tree([])
    assert not oracle.is_valid_tree([-1] + list(range(64)))


# ----------------------------------------------------------------------------- RoPE


def test_rope_two_dims_is_plane_rotation():
    x = np.array([[1.0, 0.0], [0.0, 1.0], [2.0, -3.0]])
    pos = np.array([1, 2, 5])
    y = oracle.rope_rotate_half(x, pos)
    for r in range(3):
        c, s = math.cos(pos[r]), math.sin(pos[r])
        assert y[r, 0] == pytest.approx(x[r, 0] * c - x[r, 1] * s, abs=1e-15)
        assert y[r, 1] == pytest.approx(x[r, 1] * c + x[r, 0] * s, abs=1e-15)


def test_rope_second_frequency_and_pairing():
    # D = 4: pairs are (0,2) and (1,3); the second pair turns by pos * 10000^(-1/2).
    x = np.array([[0.0, 1.0, 0.0, 0.0]])
    y = oracle.rope_rotate_half(x, np.array([7]))
    assert y[0, 0] == 0.0 and y[0, 2] == 0.0
    assert y[0, 1] == pytest.approx(math.cos(0.07), abs=1e-15)
    assert y[0, 3] == pytest.approx(math.sin(0.07), abs=1e-15)


def test_rope_identity_norm_and_relative_property():
    rng = np.random.default_rng(3)
    q = rng.standard_normal((1, 128))
    k = rng.standard_normal((1, 128))
    assert np.array_equal(oracle.rope_rotate_half(q, np.array([0])), q)
    assert np.linalg.norm(oracle.rope_rotate_half(q, np.array([977]))) == pytest.approx(
        np.linalg.norm(q), rel=1e-13)
    d1 = oracle.rope_rotate_half(q, np.array([5])) @ oracle.rope_rotate_half(k, np.array([3])).T
    d2 = oracle.rope_rotate_half(q, np.array([3012])) @ oracle.rope_rotate_half(k, np.array([3010])).T
    assert d1[0, 0] == pytest.approx(d2[0, 0], abs=1e-9)
    d3 = oracle.rope_rotate_half(q, np.array([5])) @ oracle.rope_rotate_half(k, np.array([4])).T
    assert abs(d3[0, 0] - d1[0, 0]) > 1e-6


# ----------------------------------------------------------------------------- attention


def _python_attention(q, k, v, allowed_fn, scale):
    """Pure-Python loops with math.exp: the definition, element by element."""
    T, D = len(q), len(q[0])
    out = [[0.0] * D for _ in range(T)]
    for i in range(T):
        js = [j for j in range(len(k)) if allowed_fn(i, j)]
        if not js:
            continue
        s = [sum(q[i][d] * k[j][d] for d in range(D)) * scale for j in js]
        mx = max(s)
        w = [math.exp(x - mx) for x in s]
        z = sum(w)
        for idx, j in enumerate(js):
            for d in range(D):
                out[i][d] += w[idx] / z * v[j][d]
    return np.array(out)


def test_bruteforce_python_loops_on_tiny_random_tree():
    rng = np.random.default_rng(11)
    parent = wl.config1_tree(rng, T=9, max_depth=3, max_children=3)
    T, P, D = 9, 5, 8
    q = _rand_f64_from_bf16(rng, (T, D))
    k = _rand_f64_from_bf16(rng, (P + T + 3, D))
    v = _rand_f64_from_bf16(rng, (P + T + 3, D))
    mask = oracle.tree_mask_bits(parent)

    def is_ancestor_or_self(t, i):
        while i >= 0:
            if i == t:
                return True
            i = int(parent[i])
        return False

    def allowed(i, j):
        return j < P or (P <= j < P + T and is_ancestor_or_self(j - P, i))

    ref = _python_attention(q.tolist(), k.tolist(), v.tolist(), allowed, 1.0 / math.sqrt(D))
    got = oracle.tree_attn(q, k, v, P, mask)
    assert np.abs(got - ref).max() < 1e-13


@pytest.mark.parametrize("P,T,D", [(23, 9, 16), (0, 6, 8), (70, 64, 128)])
def test_chain_tree_equals_causal_attention_with_positions(P, T, D):
    """A chain-shaped tree is an ordinary continuation: with RoPE at positions P + depth
    it must equal causal attention over the P + T tokens at positions 0..P+T-1."""
    rng = np.random.default_rng(100 + P)
    n = P + T
    q_all = _rand_f64_from_bf16(rng, (n, D))
    k_all = _rand_f64_from_bf16(rng, (n, D))
    v_all = _rand_f64_from_bf16(rng, (n, D))
    pos_all = np.arange(n)
    causal = oracle.causal_attn_textbook(oracle.rope_rotate_half(q_all, pos_all),
                                         oracle.rope_rotate_half(k_all, pos_all), v_all)
    parent = wl.chain_tree(T)
    pos_tree = oracle.tree_positions(parent, P)
    q_tree = oracle.rope_rotate_half(q_all[P:], pos_tree)
    k_cache = np.concatenate([oracle.rope_rotate_half(k_all[:P], np.arange(P)),
                              oracle.rope_rotate_half(k_all[P:], pos_tree)])
    got = oracle.tree_attn(q_tree, k_cache, v_all, P, oracle.tree_mask_bits(parent))
    assert np.abs(got - causal[P:]).max() < 1e-12


def test_single_node_tree_equals_one_token_decode():
    rng = np.random.default_rng(5)
    P, D = 37, 32
    q = _rand_f64_from_bf16(rng, (1, D))
    k = _rand_f64_from_bf16(rng, (P + 1, D))
    v = _rand_f64_from_bf16(rng, (P + 1, D))
    s = [sum(q[0, d] * k[j, d] for d in range(D)) / math.sqrt(D) for j in range(P + 1)]
    mx = max(s)
    w = [math.exp(x - mx) for x in s]
    ref = sum(w[j] * v[j] for j in range(P + 1)) / sum(w)
    got = oracle.tree_attn(q, k, v, P, oracle.tree_mask_bits(wl.single_node_tree()))
    assert np.abs(got[0] - ref).max() < 1e-13


def test_uniform_closed_forms_read_back_the_mask():
    """q = 0 makes the softmax uniform over visible keys, so outputs are counts."""
    rng = np.random.default_rng(9)
    parent = wl.eagle2_like_tree(rng, T=60, max_depth=6)
    T, D = 60, 16
    depth = oracle.tree_depth(parent)
    mask = oracle.tree_mask_bits(parent)
    for P in (0, 1, 77, 640):
        q = np.zeros((T, D))
        k = rng.standard_normal((P + T + 4, D))
        v = np.zeros((P + T + 4, D))
        v[P:P + T] = 1.0
        v[P + T:] = 1e9                                   # beyond the tree: never visible
        out = oracle.tree_attn(q, k, v, P, mask)
        for i in range(T):
            assert out[i, 0] == pytest.approx((depth[i] + 1) / (P + depth[i] + 1), rel=1e-14)
        for t in (0, 1, 17, 59):
            v[:] = 0.0
            v[P + t] = 1.0
            out = oracle.tree_attn(q, k, v, P, mask)
            for i in range(T):
                is_anc = (int(mask[i]) >> t) & 1
                assert out[i, 3] == pytest.approx(is_anc / (P + depth[i] + 1), rel=1e-14)


def test_poisoned_invisible_slots_do_not_leak():
    rng = np.random.default_rng(21)
    parent = wl.config1_tree(rng, T=26, max_depth=5)
    T, P, D = 26, 50, 32
    mask = oracle.tree_mask_bits(parent)
    q = _rand_f64_from_bf16(rng, (T, D))
    k = _rand_f64_from_bf16(rng, (P + T + 8, D))
    v = _rand_f64_from_bf16(rng, (P + T + 8, D))
    clean = oracle.tree_attn(q, k, v, P, mask)
    k2, v2 = k.copy(), v.copy()
    k2[P + T:] = np.nan
    v2[P + T:] = np.inf
    out = oracle.tree_attn(q, k2, v2, P, mask)
    assert np.array_equal(out, clean)
    # a leaf's row is invisible to every other node: poisoning it changes only that node
    leaf = T - 1
    assert all(parent[i] != leaf for i in range(T))
    k3, v3 = k.copy(), v.copy()
    k3[P + leaf] = 1e4
    v3[P + leaf] = -1e4
    out = oracle.tree_attn(q, k3, v3, P, mask)
    keep = np.arange(T) != leaf
    assert np.array_equal(out[keep], clean[keep])
    assert not np.allclose(out[leaf], clean[leaf])


def test_peaked_softmax_hits_ancestor_only():
    rng = np.random.default_rng(22)
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    T, P, D = 5, 12, 64
    mask = oracle.tree_mask_bits(parent)
    q = rng.standard_normal((T, D))
    k = rng.standard_normal((P + T, D)) * 0.01
    v = rng.standard_normal((P + T, D))
    k[P + 1] = 40.0 * q[3]          # node 1 is node 3's parent: node 3 locks onto it
    k[P + 2] = 40.0 * q[3]          # node 2 is not an ancestor of node 3: must be ignored
    out = oracle.tree_attn(q, k, v, P, mask)
    assert np.abs(out[3] - v[P + 1]).max() < 1e-9


def test_invariance_prefix_permutation_and_tree_relabelling():
    rng = np.random.default_rng(31)
    parent = wl.config1_tree(rng, T=12, max_depth=4)
    T, P, D = 12, 40, 32
    q = _rand_f64_from_bf16(rng, (T, D))
    k = _rand_f64_from_bf16(rng, (P + T, D))
    v = _rand_f64_from_bf16(rng, (P + T, D))
    base = oracle.tree_attn(q, k, v, P, oracle.tree_mask_bits(parent))
    perm = rng.permutation(P)
    kp, vp = k.copy(), v.copy()
    kp[:P], vp[:P] = k[perm], v[perm]
    assert np.abs(oracle.tree_attn(q, kp, vp, P, oracle.tree_mask_bits(parent)) - base).max() < 1e-12
    # relabel nodes by another parent<child order: reverse order inside each depth level
    depth = oracle.tree_depth(parent)
    order = sorted(range(T), key=lambda i: (depth[i], -i))
    new_of_old = {o: n for n, o in enumerate(order)}
    parent2 = np.array([-1 if parent[o] < 0 else new_of_old[parent[o]] for o in order], dtype=np.int32)
    assert oracle.is_valid_tree(parent2)
    q2 = q[order]
    k2, v2 = k.copy(), v.copy()
    k2[P:], v2[P:] = k[P:][order], v[P:][order]
    out2 = oracle.tree_attn(q2, k2, v2, P, oracle.tree_mask_bits(parent2))
    assert np.abs(out2 - base[order]).max() < 1e-12


def test_convexity_weights_sum_to_one_and_bounds():
    rng = np.random.default_rng(41)
    parent = wl.eagle2_like_tree(rng, T=60, max_depth=6)
    T, P, D = 60, 333, 16
    mask = oracle.tree_mask_bits(parent)
    q = 3.0 * rng.standard_normal((T, D))
    k = rng.standard_normal((P + T, D))
    v = rng.standard_normal((P + T, D))
    ones = oracle.tree_attn(q, k, np.ones((P + T, D)), P, mask)
    assert np.abs(ones - 1.0).max() < 1e-14
    out = oracle.tree_attn(q, k, v, P, mask)
    assert (out <= v.max(axis=0) + 1e-12).all() and (out >= v.min(axis=0) - 1e-12).all()


def test_no_visible_key_gives_zero_row_and_scale_is_used():
    q = np.ones((2, 4))
    k = np.arange(8.0).reshape(2, 4)
    v = np.ones((2, 4))
    out = oracle.tree_attn(q, k, v, 0, np.array([0, 3], dtype=np.uint64))
    assert np.array_equal(out[0], np.zeros(4))
    # scale: two keys with score gap g: weights are sigmoid(scale * g)
    v = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]])
    g = float(q[1] @ (k[1] - k[0]))
    for scale in (0.5, 0.125):
        out = oracle.tree_attn(q, k, v, 0, np.array([1, 3], dtype=np.uint64), scale=scale)
        assert out[1, 1] == pytest.approx(1.0 / (1.0 + math.exp(-scale * g)), rel=1e-12)
    out = oracle.tree_attn(q, k, v, 0, np.array([1, 3], dtype=np.uint64))
    assert out[1, 1] == pytest.approx(1.0 / (1.0 + math.exp(-g / 2.0)), rel=1e-12)


def test_bf16_conversions_roundtrip_and_rne():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)          # finite positives
    f = oracle.bf16_bits_to_f64(bits)
    assert np.array_equal(oracle.f64_to_bf16_bits(f), bits)
    assert np.array_equal(wl.bf16_bits_from_f32(f.astype(np.float32)), bits)
    # 1 + 2^-8 lies halfway between bf16 neighbours 1.0 (even) and 1 + 2^-7: ties to even
    assert int(oracle.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0]) == 0x3F80
    assert int(oracle.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0]) == 0x3F82
    assert oracle.bf16_bits_to_f64(np.array([0x3F80, 0xC000], dtype=np.uint16)).tolist() == [1.0, -2.0]
    q = wl.normal_bf16_bits(np.random.default_rng(0), (4, 8))
    a = tree_attn_bits(q[:2], q, q, 2, np.array([1, 3], dtype=np.uint64))
    b = oracle.tree_attn(oracle.bf16_bits_to_f64(q[:2]), oracle.bf16_bits_to_f64(q),
                         oracle.bf16_bits_to_f64(q), 2, np.array([1, 3], dtype=np.uint64))
    assert np.array_equal(a, b)
