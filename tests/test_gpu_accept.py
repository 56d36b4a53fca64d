"""GPU parity (bit-exact): tree metadata, vocabulary argmax, acceptance, KV compaction."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import bits_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


def i32(x):
    return torch.tensor(np.asarray(x), dtype=torch.int32, device="cuda")


# ----------------------------------------------------------------------------- tree_build


def test_tree_build_matches_oracle():
    rng = np.random.default_rng(1)
    trees = [wl.eagle2_like_tree(rng, 60, 6) for _ in range(5)] + [wl.chain_tree(60), wl.star_tree(60)]
    prefixes = rng.integers(0, 5000, size=len(trees)).astype(np.int32)
    par = i32(np.array(trees))
    B, T = par.shape
    mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
    depth = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    pos = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_tree_build(par, i32(prefixes), mask, depth, pos, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for b, p in enumerate(trees):
        assert np.array_equal(mask[b].cpu().numpy().view(np.uint64), oracle.tree_mask_bits(p))
        assert np.array_equal(depth[b].cpu().numpy(), oracle.tree_depth(p))
        assert np.array_equal(pos[b].cpu().numpy(), oracle.tree_positions(p, prefixes[b]))


def test_tree_build_64_node_chain_and_bad_tree():
    par = i32(np.array([wl.chain_tree(64)]))
    mask = torch.zeros((1, 64), dtype=torch.int64, device="cuda")
    sv.specvlm_tree_build(par, None, mask)
    torch.cuda.synchronize()
    assert np.array_equal(mask[0].cpu().numpy().view(np.uint64), oracle.tree_mask_bits(wl.chain_tree(64)))
    bad = i32(np.array([[-1, 0, 5, 1, 2, 2]]))
    mask = torch.zeros((1, 6), dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_tree_build(bad, None, mask, status=status)
    torch.cuda.synchronize()
    assert status.item() & sv.STATUS_BAD_TREE
    assert mask[0].cpu().tolist() == [1 << i for i in range(6)]


# ----------------------------------------------------------------------------- argmax


def gpu_argmax(logits_np):
    lg = torch.from_numpy(logits_np).cuda()
    out = torch.full(lg.shape[:2], -7, dtype=torch.int32, device="cuda")
    sv.specvlm_argmax(lg, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("V", [32000, 32001, 4, 1, 7, 2048 * 4 + 12, 151936])
def test_argmax_matches_oracle_bit_exact(V):
    rng = np.random.default_rng(V)
    x = rng.standard_normal((2, 5, V), dtype=np.float32)
    if V % 4:   # rows must start 16-byte aligned: pad the row stride
        Vp = (V + 3) // 4 * 4
        store = torch.zeros((2, 5, Vp), dtype=torch.float32, device="cuda")
        store[:, :, :V] = torch.from_numpy(x).cuda()
        store[:, :, V:] = 1e30                       # padding must never win
        out = torch.zeros((2, 5), dtype=torch.int32, device="cuda")
        sv.specvlm_argmax(store[:, :, :V], out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
    else:
        got = gpu_argmax(x)
    assert np.array_equal(got, oracle.vocab_argmax(x))


def test_argmax_more_rows_than_one_grid_dimension_holds():
    """B * T > 65535 rows: rows are laid along grid x, which has no such limit."""
    rng = np.random.default_rng(65536)
    x = rng.standard_normal((1100, 60, 64), dtype=np.float32)
    assert np.array_equal(gpu_argmax(x), oracle.vocab_argmax(x))


def test_argmax_tie_rules():
    V = 32000
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 8, V), dtype=np.float32)
    x[0, 0, 31999] = x[0, 0, 12345] = x[0, 0, 777] = 9.0          # equal maxima: lowest index
    x[0, 1, 0] = 9.0
    x[0, 2, V - 1] = 9.0
    x[0, 3, :] = -0.0
    x[0, 3, 9999] = 0.0                                            # -0 == +0: index 0
    x[0, 4, :] = -np.inf                                           # all -inf: index 0
    x[0, 5, :] = 3.0                                               # constant row: index 0
    x[0, 6, :] = -np.inf
    x[0, 6, 20001] = -1e30
    x[0, 7, 4096] = np.inf
    got = gpu_argmax(x)
    assert got[0].tolist() == [777, 0, V - 1, 0, 0, 0, 20001, 4096]
    assert np.array_equal(got, oracle.vocab_argmax(x))


# ----------------------------------------------------------------------------- accept


def gpu_accept(draft, parent, target_tokens=None, logits=None, acc_stride=8):
    B, T = np.asarray(draft).shape
    tok = i32(target_tokens) if target_tokens is not None else torch.zeros((B, T), dtype=torch.int32, device="cuda")
    lg = torch.from_numpy(logits).cuda() if logits is not None else None
    idx = torch.full((B, acc_stride), -99, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -99, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -99, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_accept(i32(draft), i32(parent), lg, tok, idx, n, nxt, status)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), n.cpu().numpy(), nxt.cpu().numpy(), tok.cpu().numpy(), status.item()


def expected_accept(parents, drafts, targets, acc_stride):
    B = len(parents)
    idx = np.full((B, acc_stride), -1, dtype=np.int32)
    n = np.zeros(B, dtype=np.int32)
    nxt = np.zeros(B, dtype=np.int32)
    for b in range(B):
        path, n[b], nxt[b] = oracle.accept_topdown(parents[b], drafts[b], targets[b])
        assert (path, n[b], nxt[b]) == oracle.accept_bruteforce(parents[b], drafts[b], targets[b])
        m = min(len(path), acc_stride)
        idx[b, :m] = path[:m]
    return idx, n, nxt


def test_accept_small_vocab_random_trees_bit_exact():
    rng = np.random.default_rng(4)
    B, T = 64, 60
    parents = np.array([wl.eagle2_like_tree(rng, T, 6) for _ in range(B)])
    drafts = rng.integers(0, 3, size=(B, T)).astype(np.int32)      # forces matches and duplicate siblings
    targets = rng.integers(0, 3, size=(B, T)).astype(np.int32)
    idx, n, nxt, _, status = gpu_accept(drafts, parents, targets, acc_stride=8)
    e_idx, e_n, e_nxt = expected_accept(parents, drafts, targets, 8)
    assert status == 0
    assert np.array_equal(idx, e_idx) and np.array_equal(n, e_n) and np.array_equal(nxt, e_nxt)
    assert n.max() >= 3 and n.min() == 0


@pytest.mark.parametrize("T", [1, 2, 26, 64])
def test_accept_shapes_chain_and_truncated_stride(T):
    rng = np.random.default_rng(T)
    parents = np.array([wl.chain_tree(T), wl.star_tree(T)])
    drafts = rng.integers(0, 2, size=(2, T)).astype(np.int32)
    targets = rng.integers(0, 2, size=(2, T)).astype(np.int32)
    drafts[0, 1:] = targets[0, :-1]                                # chain fully accepted: depth T-1
    for stride in (1, 4, 64):
        idx, n, nxt, _, status = gpu_accept(drafts, parents, targets, acc_stride=stride)
        e_idx, e_n, e_nxt = expected_accept(parents, drafts, targets, stride)
        assert status == 0 and n[0] == T - 1
        assert np.array_equal(idx, e_idx) and np.array_equal(n, e_n) and np.array_equal(nxt, e_nxt)


def test_accept_from_logits_with_planted_paths():
    cfg = wl.get_config("cfg2")
    rng = np.random.default_rng(cfg.seed)
    B = 7
    parents, drafts, logits, paths = [], [], [], []
    for b in range(B):
        p = wl.eagle2_like_tree(rng, cfg.T, cfg.max_depth)
        d = wl.sibling_distinct_tokens(rng, p, cfg.V)
        lg, path = wl.planted_logits(rng, p, d, cfg.V, plant_len=b)     # lengths 0..6
        parents.append(p), drafts.append(d), logits.append(lg), paths.append(path)
    logits = np.stack(logits)
    idx, n, nxt, tok, status = gpu_accept(np.array(drafts), np.array(parents), logits=logits, acc_stride=7)
    assert status == 0
    targets = oracle.vocab_argmax(logits)
    assert np.array_equal(tok, targets)
    e_idx, e_n, e_nxt = expected_accept(parents, drafts, targets, 7)
    assert np.array_equal(idx, e_idx) and np.array_equal(n, e_n) and np.array_equal(nxt, e_nxt)
    assert n.tolist() == list(range(B))
    for b in range(B):
        assert idx[b, :n[b] + 1].tolist() == paths[b]


def test_accept_fully_rejected_and_bad_tree():
    parents = np.array([wl.star_tree(6), [-1, 0, 3, 1, 2, 2]])
    drafts = np.array([[5, 10, 11, 12, 13, 14]] * 2, dtype=np.int32)
    targets = np.array([[99, 1, 2, 3, 4, 5]] * 2, dtype=np.int32)
    idx, n, nxt, _, status = gpu_accept(drafts, parents, targets, acc_stride=4)
    assert idx.tolist() == [[0, -1, -1, -1]] * 2 and n.tolist() == [0, 0] and nxt.tolist() == [99, 99]
    assert status & sv.STATUS_BAD_TREE


# ----------------------------------------------------------------------------- compaction


def make_cache(rng, L, B, H, S_cap, guard=2):
    """K and V stores with guard slots before and after every (l, b, h) slab."""
    store = wl.normal_bf16_bits(rng, (2, L, B, H, S_cap + 2 * guard, 128))
    return store


def run_compaction(fused, rng, L, B, H, T, prefixes, parents, drafts, targets):
    guard = 2
    S_cap = int(max(prefixes)) + T
    store = make_cache(rng, L, B, H, S_cap, guard)
    t_store = bits_to_torch(store)
    k = t_store[0][:, :, :, guard:guard + S_cap, :]
    v = t_store[1][:, :, :, guard:guard + S_cap, :]
    acc_stride = 8
    e_idx, e_n, e_nxt = expected_accept(parents, drafts, targets, acc_stride)
    full_idx, _, _ = expected_accept(parents, drafts, targets, 64)
    ek, ev, e_new = oracle.kv_compact(store[0][:, :, :, guard:guard + S_cap], store[1][:, :, :, guard:guard + S_cap],
                                      prefixes, full_idx, e_n)
    expect = store.copy()
    expect[0][:, :, :, guard:guard + S_cap] = ek
    expect[1][:, :, :, guard:guard + S_cap] = ev
    pl = i32(prefixes)
    new_pl = torch.full((B,), -5, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if fused:
        idx = torch.full((B, acc_stride), -99, dtype=torch.int32, device="cuda")
        n = torch.full((B,), -99, dtype=torch.int32, device="cuda")
        nxt = torch.full((B,), -99, dtype=torch.int32, device="cuda")
        sv.specvlm_accept_compact(i32(drafts), i32(parents), i32(targets), k, v, pl, idx, n, nxt, new_pl, status)
        torch.cuda.synchronize()
        assert np.array_equal(idx.cpu().numpy(), e_idx)
        assert np.array_equal(n.cpu().numpy(), e_n) and np.array_equal(nxt.cpu().numpy(), e_nxt)
    else:
        sv.specvlm_kv_compact(k, v, pl, i32(full_idx), i32(e_n), new_pl, status)
        torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(new_pl.cpu().numpy(), e_new)
    assert np.array_equal(pl.cpu().numpy(), prefixes)
    assert np.array_equal(torch_to_bits(t_store), expect), "cache bytes differ from the oracle (incl. guards)"
    return e_n


@pytest.mark.parametrize("fused", [False, True])
def test_compaction_whole_buffer_bit_exact(fused):
    rng = np.random.default_rng(6)
    L, B, H, T = 3, 5, 4, 60
    parents = np.array([wl.eagle2_like_tree(rng, T, 6) for _ in range(B)])
    drafts = rng.integers(0, 2, size=(B, T)).astype(np.int32)
    targets = rng.integers(0, 2, size=(B, T)).astype(np.int32)
    prefixes = np.array([17, 300, 0, 64, 255], dtype=np.int32)
    n = run_compaction(fused, rng, L, B, H, T, prefixes, parents, drafts, targets)
    assert n.max() >= 2


@pytest.mark.parametrize("fused", [False, True])
def test_compaction_long_chain_fully_accepted_and_hazard(fused):
    """A 64-node chain accepted to the end is the identity; a sparse path has overlapping
    source and destination slots."""
    rng = np.random.default_rng(7)
    T = 64
    chain = wl.chain_tree(T)
    # sparse path 0 -> 2 -> 5 -> 9 -> ... : parent of node t_k is t_{k-1}; other nodes hang off the root
    sparse = np.zeros(T, dtype=np.int32)
    sparse[0] = -1
    path = [0, 2, 5, 9, 14, 20, 27, 35, 44, 54]
    for a, b in zip(path[:-1], path[1:]):
        sparse[b] = a
    parents = np.array([chain, sparse])
    drafts = np.arange(T, dtype=np.int32)[None, :].repeat(2, 0) + 100
    targets = np.full((2, T), 7, dtype=np.int32)
    for b, par in enumerate(parents):
        for i in range(1, T):
            if b == 0 or i in path:
                targets[b, par[i]] = drafts[b, i]
    prefixes = np.array([33, 128], dtype=np.int32)
    n = run_compaction(fused, rng, 2, 2, 3, T, prefixes, parents, drafts, targets)
    assert n.tolist() == [63, 9]


def test_kv_compact_rejects_bad_accept_data_without_touching_the_cache():
    rng = np.random.default_rng(8)
    L, B, H, S_cap = 1, 2, 2, 100
    store = wl.normal_bf16_bits(rng, (2, L, B, H, S_cap, 128))
    t_store = bits_to_torch(store)
    pl = i32([10, 10])
    idx = i32([[0, 3, 2, -1], [0, 1, 2, -1]])        # sequence 0: not increasing
    n = i32([2, 2])
    new_pl = torch.zeros(2, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.specvlm_kv_compact(t_store[0], t_store[1], pl, idx, n, new_pl, status)
    torch.cuda.synchronize()
    assert status.item() & sv.STATUS_BAD_ACCEPT
    assert new_pl.tolist() == [10, 13]
    assert np.array_equal(torch_to_bits(t_store), store)          # seq 1 was the identity move
    with pytest.raises(sv.SpecvlmError):
        sv.specvlm_kv_compact(t_store[0], t_store[1], pl, idx, n, pl, status)   # aliasing
