"""GPU parity: specvlm_tree_verify_attn (through the C ABI) against the fp64 CPU oracle."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import (ATTN_MAX_ABS, ATTN_MEAN_ABS, assert_attn_close, bits_to_torch, mask_to_torch,
                  oracle_attn_all, torch_to_bits)

pytestmark = pytest.mark.gpu

# Every test in this file runs on each kernel variant, selected through the descriptor flags:
# the whole-SM tcgen05 configuration (default), the half-SM tcgen05 configuration used for
# launches declared independent of their predecessor, and the legacy mma.sync kernels.
ATTN_FLAGS = 0


@pytest.fixture(autouse=True, params=[0, sv.ATTN_FLAG_INPUTS_STABLE, sv.ATTN_FLAG_PREFIX_STABLE, sv.ATTN_FLAG_PREFIX_STABLE | sv.ATTN_FLAG_HALF_SM,
                        sv.ATTN_FLAG_LEGACY_MMA],
                ids=["tcgen05_full_sm", "tcgen05_half_sm", "tcgen05_prefix_prefetch", "tcgen05_half_sm_prefix_prefetch", "legacy_mma"])
def _attn_path(request):
    global ATTN_FLAGS
    ATTN_FLAGS = request.param
    yield
    ATTN_FLAGS = 0


def run_attn(q_bits, k_bits, v_bits, prefix_len, masks=None, parents=None, num_splits=0, scale=0.0,
             out_fill=None):
    """Marshal numpy inputs, call the library, return (out bits [B][H][T][D], status)."""
    q = bits_to_torch(q_bits)
    k = bits_to_torch(k_bits)
    v = bits_to_torch(v_bits)
    out = torch.empty_like(q)
    if out_fill is not None:
        out.fill_(out_fill)
    pl = torch.tensor(np.asarray(prefix_len), dtype=torch.int32, device="cuda")
    mk = mask_to_torch(np.asarray(masks)) if masks is not None else None
    par = torch.tensor(np.asarray(parents), dtype=torch.int32, device="cuda") if parents is not None else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    desc = sv.make_attn_desc(q, k, v, out, num_splits, scale, ATTN_FLAGS)
    ws = sv.alloc_attn_workspace(desc, q.device)
    sv.specvlm_tree_verify_attn(q, k, v, pl, par, mk, out, workspace=ws, status=status, desc=desc)
    torch.cuda.synchronize()
    # the workspace must be left ready for the next call: run again and compare bytes
    out2 = torch.empty_like(q)
    desc2 = sv.make_attn_desc(q, k, v, out2, num_splits, scale, ATTN_FLAGS)
    sv.specvlm_tree_verify_attn(q, k, v, pl, par, mk, out2, workspace=ws, status=status, desc=desc2)
    torch.cuda.synchronize()
    a, b = torch_to_bits(out), torch_to_bits(out2)
    assert np.array_equal(a, b), "second call on the same workspace differs"
    return a, int(status.item())


def make_case(seed, B, H, T, prefixes, tree="eagle", slack=0, D=128):
    rng = np.random.default_rng(seed)
    S_cap = int(max(prefixes)) + T + slack
    parents, masks = [], []
    for b in range(B):
        if tree == "chain":
            p = wl.chain_tree(T)
        elif tree == "star":
            p = wl.star_tree(T)
        elif T >= 20:
            p = wl.eagle2_like_tree(rng, T=T, max_depth=min(6, T - 1))
        else:
            p = wl.config1_tree(rng, T=T, max_depth=min(4, T - 1)) if T > 1 else wl.single_node_tree()
        parents.append(p)
        masks.append(oracle.tree_mask_bits(p))
    q = wl.normal_bf16_bits(rng, (B, H, T, D))
    k = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    v = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    return q, k, v, np.array(prefixes, dtype=np.int32), np.array(parents), np.array(masks)


def test_config1_all_heads_matches_oracle():
    cfg = wl.get_config("cfg1")
    rng = np.random.default_rng(cfg.seed)
    parent = wl.config1_tree(rng, T=cfg.T, max_depth=cfg.max_depth)
    mask = oracle.tree_mask_bits(parent)
    q = wl.normal_bf16_bits(rng, (1, cfg.H, cfg.T, cfg.D))
    k = wl.normal_bf16_bits(rng, (1, cfg.H, cfg.s_cap, cfg.D))
    v = wl.normal_bf16_bits(rng, (1, cfg.H, cfg.s_cap, cfg.D))
    ref = oracle_attn_all(q, k, v, [cfg.prefix_nominal], [mask])
    got, status = run_attn(q, k, v, [cfg.prefix_nominal], masks=[mask])
    assert status == 0
    assert_attn_close(got, ref)
    # mask derived inside the kernel from the parent array gives the same bytes
    got2, status = run_attn(q, k, v, [cfg.prefix_nominal], parents=[parent])
    assert status == 0 and np.array_equal(got, got2)


@pytest.mark.parametrize("T", [1, 7, 16, 17, 26, 33, 60, 64])
@pytest.mark.parametrize("P", [0, 1, 63, 64, 65, 200])
def test_shapes_and_ragged_tails(T, P):
    q, k, v, pl, parents, masks = make_case(1000 * T + P, B=1, H=3, T=T, prefixes=[P], slack=5)
    ref = oracle_attn_all(q, k, v, pl, masks)
    for splits in (1, 3):
        got, status = run_attn(q, k, v, pl, masks=masks, num_splits=splits)
        assert status == 0
        assert_attn_close(got, ref)


@pytest.mark.parametrize("splits", [0, 1, 2, 5, 7, 64])
def test_ragged_batch_and_split_counts(splits):
    prefixes = [640, 5, 0, 333, 129, 1000, 64, 777]
    q, k, v, pl, parents, masks = make_case(77, B=8, H=4, T=60, prefixes=prefixes, slack=64)
    ref = oracle_attn_all(q, k, v, pl, masks)
    got, status = run_attn(q, k, v, pl, masks=masks, num_splits=splits)
    assert status == 0
    assert_attn_close(got, ref)


def test_split_invariance():
    q, k, v, pl, parents, masks = make_case(5, B=2, H=4, T=60, prefixes=[1500, 900])
    base, _ = run_attn(q, k, v, pl, masks=masks, num_splits=1)
    for splits in (2, 6, 13):
        got, _ = run_attn(q, k, v, pl, masks=masks, num_splits=splits)
        d = np.abs(oracle.bf16_bits_to_f64(got) - oracle.bf16_bits_to_f64(base))
        assert d.max() <= 2e-3


def test_uniform_scores_read_back_every_mask_bit():
    """q = 0: every visible key gets the same weight, so the output counts visible rows."""
    rng = np.random.default_rng(8)
    T, H, D = 60, 2, 128
    parent = wl.eagle2_like_tree(rng, T=T, max_depth=6)
    mask = oracle.tree_mask_bits(parent)
    depth = oracle.tree_depth(parent)
    for P in (0, 100, 131):
        S_cap = P + T + 7
        q = np.zeros((1, H, T, D), dtype=np.uint16)
        k = wl.normal_bf16_bits(rng, (1, H, S_cap, D))
        one = wl.bf16_bits_from_f32(np.array([1.0], dtype=np.float32))[0]
        # column block t of V marks tree slot t: V[P + t][2t .. 2t+1] = 1
        v = np.zeros((1, H, S_cap, D), dtype=np.uint16)
        for t in range(T):
            v[0, :, P + t, 2 * t:2 * t + 2] = one
        v[0, :, P + T:, :] = one                           # beyond the tree: must stay invisible
        got, status = run_attn(q, k, v, [P], masks=[mask], num_splits=2)
        assert status == 0
        out = oracle.bf16_bits_to_f64(got)
        for i in range(T):
            denom = P + depth[i] + 1
            for t in range(T):
                want = ((int(mask[i]) >> t) & 1) / denom
                want = oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(np.array([want])))[0]
                assert abs(out[0, 0, i, 2 * t] - want) <= 2.0 ** -8 * want + 1e-30, (P, i, t)
                assert abs(out[0, 1, i, 2 * t + 1] - want) <= 2.0 ** -8 * want + 1e-30
            assert (out[0, :, i, 2 * T:] == 0).all()


def test_poisoned_slots_never_leak():
    """Slots beyond the tree hold NaN / Inf patterns (an uninitialised cache); tree slots of
    non-ancestors hold huge finite values; rows >= T of nothing. None may reach the output."""
    rng = np.random.default_rng(13)
    B, H, T, D = 2, 3, 26, 128
    prefixes = [70, 301]
    S_cap = max(prefixes) + T + 40
    parents = [wl.config1_tree(rng, T=T, max_depth=5) for _ in range(B)]
    masks = [oracle.tree_mask_bits(p) for p in parents]
    q = wl.normal_bf16_bits(rng, (B, H, T, D))
    k = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    v = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    clean = oracle_attn_all(q, k, v, prefixes, masks)
    nan, pinf, ninf = 0x7FC0, 0x7F80, 0xFF80
    for b, P in enumerate(prefixes):
        k[b, :, P + T:, 0::3] = nan
        k[b, :, P + T:, 1::3] = pinf
        k[b, :, P + T:, 2::3] = ninf
        v[b, :, P + T:, 0::2] = nan
        v[b, :, P + T:, 1::2] = ninf
    ref = oracle_attn_all(q, k, v, prefixes, masks)
    assert np.array_equal(ref, clean)
    for splits in (1, 4):
        got, status = run_attn(q, k, v, prefixes, masks=masks, num_splits=splits)
        assert status == 0
        assert_attn_close(got, ref)
    # a leaf's slot is visible to that leaf only: poison it with large finite values
    big = wl.bf16_bits_from_f32(np.array([1e4, -1e4], dtype=np.float32))
    for b, P in enumerate(prefixes):
        leaf = T - 1
        k[b, :, P + leaf, :] = big[0]
        v[b, :, P + leaf, :] = big[1]
    ref2 = oracle_attn_all(q, k, v, prefixes, masks)
    got, _ = run_attn(q, k, v, prefixes, masks=masks, num_splits=3)
    keep = np.arange(T) != T - 1
    assert_attn_close(got[:, :, keep], ref2[:, :, keep])
    assert np.array_equal(ref2[:, :, keep], clean[:, :, keep])


def test_peaked_softmax_on_ancestor_and_non_ancestor():
    rng = np.random.default_rng(14)
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    T, P, H, D = 5, 90, 2, 128
    mask = oracle.tree_mask_bits(parent)
    qf = rng.standard_normal((1, H, T, D)).astype(np.float32)
    kf = (0.01 * rng.standard_normal((1, H, P + T, D))).astype(np.float32)
    kf[0, :, P + 1] = 4.0 * qf[0, :, 3]         # ancestor of node 3: takes all its weight
    kf[0, :, P + 2] = 4.0 * qf[0, :, 3]         # not an ancestor of node 3
    q, k = wl.bf16_bits_from_f32(qf), wl.bf16_bits_from_f32(kf)
    v = wl.normal_bf16_bits(rng, (1, H, P + T, D))
    ref = oracle_attn_all(q, k, v, [P], [mask])
    got, _ = run_attn(q, k, v, [P], masks=[mask])
    assert_attn_close(got, ref)
    vf = oracle.bf16_bits_to_f64(v)
    assert np.abs(oracle.bf16_bits_to_f64(got)[0, :, 3] - vf[0, :, P + 1]).max() < 2e-2


def test_chain_tree_is_causal_attention():
    T, P, H = 24, 150, 2
    q, k, v, pl, parents, masks = make_case(15, B=1, H=H, T=T, prefixes=[P], tree="chain")
    got, _ = run_attn(q, k, v, pl, parents=parents)
    qf, kf, vf = (oracle.bf16_bits_to_f64(x) for x in (q, k, v))
    for h in range(H):
        seq_q = np.concatenate([np.zeros((P, 128)), qf[0, h]])
        causal = oracle.causal_attn_textbook(seq_q, kf[0, h, :P + T], vf[0, h, :P + T])[P:]
        assert_attn_close(got[0, h], causal)


def test_strided_token_major_layout_and_custom_scale():
    """Caches laid out [B][S][H][D] and outputs laid out [B][T][H][D] through the strides."""
    rng = np.random.default_rng(16)
    B, H, T, D, P = 2, 4, 60, 128, 500
    S_cap = P + T
    parent = wl.eagle2_like_tree(rng, T=T, max_depth=6)
    mask = oracle.tree_mask_bits(parent)
    q = wl.normal_bf16_bits(rng, (B, H, T, D))
    k = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    v = wl.normal_bf16_bits(rng, (B, H, S_cap, D))
    scale = 0.05
    ref = oracle_attn_all(q, k, v, [P, P - 37], [mask, mask], scale)
    qt = bits_to_torch(q)
    kt = bits_to_torch(np.ascontiguousarray(k.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)   # storage [B][S][H][D]
    vt = bits_to_torch(np.ascontiguousarray(v.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    out_store = torch.zeros((B, T, H, D), dtype=torch.bfloat16, device="cuda")
    out = out_store.permute(0, 2, 1, 3)
    pl = torch.tensor([P, P - 37], dtype=torch.int32, device="cuda")
    mk = mask_to_torch(np.array([mask, mask]))
    desc = sv.make_attn_desc(qt, kt, vt, out, 3, scale, ATTN_FLAGS)
    ws = sv.alloc_attn_workspace(desc, qt.device)
    sv.specvlm_tree_verify_attn(qt, kt, vt, pl, None, mk, out, workspace=ws, desc=desc)
    torch.cuda.synchronize()
    assert_attn_close(torch_to_bits(out_store).transpose(0, 2, 1, 3), ref)


def test_bad_prefix_sets_status_and_skips_sequence():
    q, k, v, pl, parents, masks = make_case(17, B=2, H=2, T=26, prefixes=[100, 100])
    bad = np.array([100, 10 ** 6], dtype=np.int32)
    got, status = run_attn(q, k, v, bad, masks=masks, num_splits=2)
    assert status & sv.STATUS_BAD_PREFIX
    ref = oracle_attn_all(q[:1], k[:1], v[:1], [100], masks[:1])
    assert_attn_close(got[:1], ref)
    assert (got[1] == 0).all()
    got, status = run_attn(q, k, v, np.array([-3, 100], dtype=np.int32), masks=masks, num_splits=1)
    assert status & sv.STATUS_BAD_PREFIX and (got[0] == 0).all()


def test_output_rows_beyond_tree_and_neighbours_untouched():
    """Only out[b][h][0..T) is written: guard rows around the output keep their bytes."""
    rng = np.random.default_rng(18)
    B, H, T, D, P = 1, 2, 26, 128, 130
    parent = wl.config1_tree(rng, T=T, max_depth=5)
    mask = oracle.tree_mask_bits(parent)
    q = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, T, D)))
    k = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, P + T, D)))
    v = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, P + T, D)))
    store = torch.full((B, H, T + 6, D), 7.0, dtype=torch.bfloat16, device="cuda")
    out = store[:, :, 3:3 + T, :]
    pl = torch.tensor([P], dtype=torch.int32, device="cuda")
    desc = sv.make_attn_desc(q, k, v, out, 2, 0.0, ATTN_FLAGS)
    ws = sv.alloc_attn_workspace(desc, q.device)
    sv.specvlm_tree_verify_attn(q, k, v, pl, None, mask_to_torch(np.array([mask])), out, workspace=ws, desc=desc)
    torch.cuda.synchronize()
    assert (store[:, :, :3] == 7.0).all() and (store[:, :, 3 + T:] == 7.0).all()
    assert not (store[:, :, 3:3 + T] == 7.0).all()


def test_invalid_arguments_are_rejected_on_the_host():
    q, k, v, pl, parents, masks = make_case(19, B=1, H=2, T=26, prefixes=[1000])
    qt, kt, vt = bits_to_torch(q), bits_to_torch(k), bits_to_torch(v)
    out = torch.empty_like(qt)
    plt = torch.tensor(pl, dtype=torch.int32, device="cuda")
    with pytest.raises(sv.SpecvlmError):       # neither mask nor parent
        sv.specvlm_tree_verify_attn(qt, kt, vt, plt, None, None, out, num_splits=1)
    with pytest.raises(sv.SpecvlmError):       # more than 8 splits without a workspace
        sv.specvlm_tree_verify_attn(qt, kt, vt, plt, None, mask_to_torch(masks), out, num_splits=12)
    with pytest.raises(sv.SpecvlmError):       # misaligned q (offset by one element)
        flat = torch.empty(qt.numel() + 8, dtype=torch.bfloat16, device="cuda")
        q_bad = flat[1:1 + qt.numel()].view_as(qt)
        sv.specvlm_tree_verify_attn(q_bad, kt, vt, plt, None, mask_to_torch(masks), out, num_splits=1)


@pytest.mark.parametrize("splits", [1, 2])
def test_late_maximum_forces_the_accumulator_rescale(splits):
    """Scores that jump by far more than 2^8 late in a CTA's key range: the output accumulator
    has to be rescaled after earlier tiles were already accumulated."""
    rng = np.random.default_rng(23)
    H, T, P, D = 2, 26, 1500, 128
    parent = wl.config1_tree(rng, T=T, max_depth=5)
    mask = oracle.tree_mask_bits(parent)
    qf = rng.standard_normal((1, H, T, D)).astype(np.float32)
    kf = (0.05 * rng.standard_normal((1, H, P + T, D))).astype(np.float32)
    for i in range(T):
        # row i finds a key aligned with it deep in the prefix, a stronger one later, and (for
        # even rows) the strongest one on its own tree slot, which is processed last
        kf[0, :, 300 + 7 * i] = 1.5 * qf[0, :, i]
        kf[0, :, 1100 + 5 * i] = 3.0 * qf[0, :, i]
        if i % 2 == 0:
            kf[0, :, P + i] = 6.0 * qf[0, :, i]
    q, k = wl.bf16_bits_from_f32(qf), wl.bf16_bits_from_f32(kf)
    v = wl.normal_bf16_bits(rng, (1, H, P + T, D))
    ref = oracle_attn_all(q, k, v, [P], [mask])
    got, status = run_attn(q, k, v, [P], masks=[mask], num_splits=splits)
    assert status == 0
    assert_attn_close(got, ref)
    vf = oracle.bf16_bits_to_f64(v)
    out = oracle.bf16_bits_to_f64(got)
    for i in range(0, T, 2):     # even rows lock onto their own tree slot
        assert np.abs(out[0, :, i] - vf[0, :, P + i]).max() < 2e-2


def test_randomized_shape_sweep():
    """Many random (batch, heads, tree size, ragged prefixes, split count) combinations."""
    rng = np.random.default_rng(1234 + ATTN_FLAGS)
    for trial in range(12):
        B = int(rng.integers(1, 4))
        H = int(rng.integers(1, 5))
        T = int(rng.integers(1, 65))
        prefixes = [int(x) for x in rng.integers(0, 900, size=B)]
        splits = int(rng.choice([0, 1, 2, 3, 4, 6, 8, 11]))
        q, k, v, pl, parents, masks = make_case(int(rng.integers(1 << 30)), B=B, H=H, T=T, prefixes=prefixes,
                                                slack=int(rng.integers(0, 70)))
        ref = oracle_attn_all(q, k, v, pl, masks)
        got, status = run_attn(q, k, v, pl, masks=masks, num_splits=splits)
        assert status == 0, (trial, B, H, T, prefixes, splits)
        assert_attn_close(got, ref)


@pytest.mark.parametrize("B,H,T", [(50, 8, 26), (23, 40, 60)])
def test_more_items_than_resident_blocks(B, H, T):
    """B * H above two blocks per SM, so the launch runs in more than one wave of blocks. Ragged
    prefixes, including empty ones and a sequence whose prefix does not fit the cache (reported,
    rows written as zeros)."""
    rng = np.random.default_rng(B * H)
    prefixes = rng.integers(0, 300, size=B)
    prefixes[3] = 0
    prefixes[B - 1] = 0
    prefixes[B // 2] = 299
    q, k, v, pl, parents, masks = make_case(4242 + B, B=B, H=H, T=T, prefixes=prefixes.tolist(), slack=3)
    ref = oracle_attn_all(q, k, v, pl, masks)
    got, status = run_attn(q, k, v, pl, masks=masks, num_splits=1)
    assert status == 0
    assert_attn_close(got, ref)
    got2, status = run_attn(q, k, v, pl, parents=parents, num_splits=1)   # masks derived in the kernel
    assert status == 0 and np.array_equal(got, got2)
    # one sequence in the middle with an impossible prefix: flagged, its rows are zeros, the rest unchanged
    bad = pl.copy()
    bad[5] = 10_000
    got3, status = run_attn(q, k, v, bad, masks=masks, num_splits=1, out_fill=7.0)
    assert status & sv.STATUS_BAD_PREFIX
    assert not got3[5].any()
    keep = np.arange(B) != 5
    assert np.array_equal(got3[keep], got[keep])


def test_invariance_under_prefix_permutation_and_tree_relabelling():
    """Properties that hold at any size: jointly permuting the prefix rows of K and V changes only
    the summation order; relabelling the tree nodes in another parent-before-child order permutes
    slots, mask bits and output rows together."""
    rng = np.random.default_rng(99)
    B, H, T, P = 1, 4, 40, 777
    q, k, v, pl, parents, masks = make_case(99, B=B, H=H, T=T, prefixes=[P])
    base, status = run_attn(q, k, v, pl, masks=masks)
    assert status == 0
    perm = rng.permutation(P)
    k2, v2 = k.copy(), v.copy()
    k2[:, :, :P] = k[:, :, perm]
    v2[:, :, :P] = v[:, :, perm]
    got, status = run_attn(q, k2, v2, pl, masks=masks)
    assert status == 0
    d = np.abs(oracle.bf16_bits_to_f64(got) - oracle.bf16_bits_to_f64(base))
    assert d.max() <= 2e-3, d.max()
    # relabel: a random order in which every parent still precedes its children
    parent = parents[0]
    depth = oracle.tree_depth(parent)
    order = np.lexsort((rng.random(T), depth))          # new label j <- old node order[j]
    assert order[0] == 0
    new_of_old = np.empty(T, dtype=np.int64)
    new_of_old[order] = np.arange(T)
    parent2 = np.array([-1] + [new_of_old[parent[order[j]]] for j in range(1, T)], dtype=np.int32)
    assert oracle.is_valid_tree(parent2)
    q3, k3, v3 = q.copy(), k.copy(), v.copy()
    q3[:, :, :] = q[:, :, order]
    k3[:, :, P:P + T] = k[:, :, P + order]
    v3[:, :, P:P + T] = v[:, :, P + order]
    got3, status = run_attn(q3, k3, v3, pl, masks=[oracle.tree_mask_bits(parent2)])
    assert status == 0
    d = np.abs(oracle.bf16_bits_to_f64(got3) - oracle.bf16_bits_to_f64(base[:, :, order]))
    assert d.max() <= 2e-3, d.max()
