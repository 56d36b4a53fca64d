"""GPU parity at the full workload sizes, in the launch configuration the benchmark times.

All L layers are launched back to back on one stream exactly as bench.py does (layer 0
waiting for its predecessor with prefix prefetch, layers 1..L-1 declared independent of the
preceding launch so that they overlap),
followed by argmax and the fused accept + compaction launch. Attention is compared with the
oracle on sampled (layer, sequence, head) outputs; argmax, acceptance and prefix lengths are
compared in full (bit-exact); compaction is compared with the oracle on sampled (layer,
sequence, head) slabs and, over the whole cache, through properties that hold at any size
(destination rows equal the pre-image source rows, every other byte unchanged).
"""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import ATTN_MAX_ABS, ATTN_MEAN_ABS, torch_to_bits

pytestmark = pytest.mark.gpu


def run_verify_step(cfg_name, sampled_layers, heads_per_layer, seed_offset=0):
    cfg = wl.get_config(cfg_name)
    dev = torch.device("cuda")
    L, B, H, T, D, V = cfg.L, cfg.B, cfg.H, cfg.T, cfg.D, cfg.V
    S_cap = cfg.s_cap
    rng = np.random.default_rng([cfg.seed, 77 + seed_offset])
    P_host = wl.draw_prefix_lens(cfg, np.random.default_rng(cfg.seed))
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    bf = dict(dtype=torch.bfloat16, device=dev)
    k_cache = torch.randn((L, B, H, S_cap, D), generator=gen, **bf)
    v_cache = torch.randn((L, B, H, S_cap, D), generator=gen, **bf)
    q = torch.randn((L, B, H, T, D), generator=gen, **bf)
    out = torch.zeros_like(q)
    # slots beyond prefix + T may hold anything in a real cache: poison them
    for b in range(B):
        k_cache[:, b, :, int(P_host[b]) + T:, :] = float("nan")
        v_cache[:, b, :, int(P_host[b]) + T:, :] = float("inf")

    parents, drafts, logits, paths = [], [], [], []
    for b in range(B):
        p = wl.eagle2_like_tree(rng, T, cfg.max_depth)
        d = wl.sibling_distinct_tokens(rng, p, V)
        lg, path = wl.planted_logits(rng, p, d, V, plant_len=int(rng.integers(0, cfg.max_depth + 1)))
        parents.append(p), drafts.append(d), logits.append(lg), paths.append(path)
    parents, drafts, logits = np.array(parents, dtype=np.int32), np.array(drafts, dtype=np.int32), np.stack(logits)
    i32 = dict(dtype=torch.int32, device=dev)
    prefix_len = torch.tensor(P_host, **i32)
    par, drf = torch.tensor(parents, **i32), torch.tensor(drafts, **i32)
    lg = torch.from_numpy(logits).to(dev)
    mask = torch.zeros((B, T), dtype=torch.int64, device=dev)
    status = torch.zeros(1, **i32)
    sv.specvlm_tree_build(par, prefix_len, mask, status=status)

    # inputs of the sampled attention outputs, copied out before compaction moves rows
    picks = []
    for l in sampled_layers:
        heads = sorted(rng.choice(H, size=min(heads_per_layer, H), replace=False).tolist())
        for b in range(B):
            for h in heads:
                n = int(P_host[b]) + T
                picks.append((l, b, h, torch_to_bits(q[l, b, h]), torch_to_bits(k_cache[l, b, h, :n]),
                              torch_to_bits(v_cache[l, b, h, :n])))
    k_before, v_before = k_cache.clone(), v_cache.clone()

    desc_ser = sv.make_attn_desc(q[0], k_cache[0], v_cache[0], out[0])   # sizes the workspace
    desc_pipe = sv.make_attn_desc(q[0], k_cache[0], v_cache[0], out[0], flags=sv.ATTN_FLAG_INPUTS_STABLE)
    desc_pipe0 = sv.make_attn_desc(q[0], k_cache[0], v_cache[0], out[0],
                                   flags=sv.ATTN_FLAG_PREFIX_STABLE | sv.ATTN_FLAG_HALF_SM)
    ws = sv.alloc_attn_workspace(desc_ser, dev)
    tok = torch.zeros((B, T), **i32)
    acc_idx = torch.zeros((B, 8), **i32)
    acc_len, nxt, new_len = torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32)
    torch.cuda.synchronize()
    for l in range(L):
        sv.specvlm_tree_verify_attn(q[l], k_cache[l], v_cache[l], prefix_len, par, mask, out[l], workspace=ws,
                                    status=status, desc=desc_pipe if l > 0 else desc_pipe0)
    sv.specvlm_argmax(lg, tok)
    sv.specvlm_accept_compact(drf, par, tok, k_cache, v_cache, prefix_len, acc_idx, acc_len, nxt, new_len, status)
    torch.cuda.synchronize()
    assert status.item() == 0

    # ---- attention on the sampled outputs
    worst_max, worst_mean = 0.0, 0.0
    masks = [oracle.tree_mask_bits(p) for p in parents]
    assert np.array_equal(mask.cpu().numpy().view(np.uint64), np.array(masks))
    for l, b, h, qb, kb, vb in picks:
        ref = oracle.attention.tree_attn_bits(qb, kb, vb, int(P_host[b]), masks[b])
        got = oracle.bf16_bits_to_f64(torch_to_bits(out[l, b, h]))
        assert np.isfinite(got).all()
        err = np.abs(got - ref)
        worst_max, worst_mean = max(worst_max, err.max()), max(worst_mean, err.mean())
    assert worst_max <= ATTN_MAX_ABS and worst_mean <= ATTN_MEAN_ABS, (worst_max, worst_mean)
    assert torch.isfinite(out.float()).all()

    # ---- argmax, acceptance, prefix lengths: everything, bit-exact
    o_tok = oracle.vocab_argmax(logits)
    assert np.array_equal(tok.cpu().numpy(), o_tok)
    e_idx = np.full((B, 8), -1, dtype=np.int32)
    e_n = np.zeros(B, dtype=np.int32)
    e_nxt = np.zeros(B, dtype=np.int32)
    for b in range(B):
        path, e_n[b], e_nxt[b] = oracle.accept_topdown(parents[b], drafts[b], o_tok[b])
        assert path == paths[b]
        e_idx[b, :len(path)] = path
    assert np.array_equal(acc_idx.cpu().numpy(), e_idx)
    assert np.array_equal(acc_len.cpu().numpy(), e_n) and np.array_equal(nxt.cpu().numpy(), e_nxt)
    assert np.array_equal(new_len.cpu().numpy(), P_host + 1 + e_n)

    # ---- compaction: oracle on sampled slabs
    seen = set()
    for l, b, h, *_ in picks:
        if (l, b, h) in seen:
            continue
        seen.add((l, b, h))
        full_idx = np.full((1, 64), -1, dtype=np.int32)
        full_idx[0, :8] = e_idx[b]
        kb = torch_to_bits(k_before[l, b, h])[None, None, None]
        vb = torch_to_bits(v_before[l, b, h])[None, None, None]
        ek, ev, _ = oracle.kv_compact(kb, vb, [int(P_host[b])], full_idx, [int(e_n[b])])
        assert np.array_equal(torch_to_bits(k_cache[l, b, h]), ek[0, 0, 0])
        assert np.array_equal(torch_to_bits(v_cache[l, b, h]), ev[0, 0, 0])
    # ---- compaction: whole-cache properties
    for cache, before in ((k_cache, k_before), (v_cache, v_before)):
        cb, bb = cache.view(torch.int16), before.view(torch.int16)
        for b in range(B):
            Pb, n = int(P_host[b]), int(e_n[b])
            assert torch.equal(cb[:, b, :, :Pb + 1], bb[:, b, :, :Pb + 1])
            assert torch.equal(cb[:, b, :, Pb + n + 1:], bb[:, b, :, Pb + n + 1:])
            for j in range(1, n + 1):
                assert torch.equal(cb[:, b, :, Pb + j], bb[:, b, :, Pb + int(e_idx[b, j])])
    return worst_max, worst_mean


def test_cfg2_llava_1_6_7b_shape():
    run_verify_step("cfg2", sampled_layers=[0, 31, 13, 22], heads_per_layer=32)


@pytest.mark.parametrize("name", ["cfg3_b1_144", "cfg3_b1_288", "cfg3_b16_144", "cfg3_b16_288"])
def test_cfg3_compressed_visual(name):
    run_verify_step(name, sampled_layers=[0, 31, 7], heads_per_layer=8)


def test_cfg4_llava_1_6_13b_shape_batch4():
    run_verify_step("cfg4", sampled_layers=[0, 39, 18], heads_per_layer=10)


def test_cfg5_video_long_prefix_batch8():
    run_verify_step("cfg5", sampled_layers=[0, 31], heads_per_layer=6)


def test_cfg1_tiny_reference_full():
    cfg = wl.get_config("cfg1")
    # config 1 uses the random-growth tree and a fixed planted length of 3
    dev = torch.device("cuda")
    rng = np.random.default_rng(cfg.seed)
    parent = wl.config1_tree(rng, T=cfg.T, max_depth=cfg.max_depth)
    draft = wl.sibling_distinct_tokens(rng, parent, cfg.V)
    logits, path = wl.planted_logits(rng, parent, draft, cfg.V, plant_len=3)
    i32 = dict(dtype=torch.int32, device=dev)
    tok = torch.zeros((1, cfg.T), **i32)
    idx = torch.zeros((1, 8), **i32)
    n, nxt = torch.zeros(1, **i32), torch.zeros(1, **i32)
    sv.specvlm_accept(torch.tensor(draft[None], **i32), torch.tensor(parent[None], **i32),
                      torch.from_numpy(logits[None]).to(dev), tok, idx, n, nxt)
    torch.cuda.synchronize()
    assert n.item() == 3 and idx[0, :4].tolist() == path
    assert nxt.item() == int(oracle.vocab_argmax(logits)[path[-1]])
