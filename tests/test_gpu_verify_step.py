"""GPU: the one-call verify step gives the same bytes as the per-call sequence, and matches the oracle."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import assert_attn_close, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("independent", [False, True])
def test_verify_step_equals_per_call_sequence_and_oracle(independent):
    rng = np.random.default_rng(11)
    L, B, H, T, V = 4, 2, 8, 60, 32000
    prefixes = np.array([700, 333], dtype=np.int32)
    S_cap = 700 + T
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    bf = dict(dtype=torch.bfloat16, device=dev)
    k = torch.randn((L, B, H, S_cap, 128), generator=gen, **bf)
    v = torch.randn((L, B, H, S_cap, 128), generator=gen, **bf)
    q = torch.randn((L, B, H, T, 128), generator=gen, **bf)
    parents, drafts, logits = [], [], []
    for b in range(B):
        p = wl.eagle2_like_tree(rng, T, 6)
        d = wl.sibling_distinct_tokens(rng, p, V)
        lg, _ = wl.planted_logits(rng, p, d, V, plant_len=3 + b)
        parents.append(p), drafts.append(d), logits.append(lg)
    i32 = dict(dtype=torch.int32, device=dev)
    par, drf = torch.tensor(np.array(parents), **i32), torch.tensor(np.array(drafts), **i32)
    lg = torch.from_numpy(np.stack(logits)).to(dev)
    pl = torch.tensor(prefixes, **i32)
    mask = torch.zeros((B, T), dtype=torch.int64, device=dev)
    sv.specvlm_tree_build(par, pl, mask)

    def fresh():
        return (k.clone(), v.clone(), torch.zeros_like(q), torch.zeros((B, T), **i32), torch.zeros((B, 8), **i32),
                torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros(1, **i32))

    k1, v1, o1, tok1, idx1, n1, nx1, nl1, st1 = fresh()
    sv.specvlm_verify_step(q, k1, v1, pl, par, mask, drf, lg, o1, tok1, idx1, n1, nx1, nl1,
                           layers_independent=independent, status=st1)
    k2, v2, o2, tok2, idx2, n2, nx2, nl2, st2 = fresh()
    for l in range(L):
        sv.specvlm_tree_verify_attn(q[l], k2[l], v2[l], pl, par, mask, o2[l], status=st2)
    sv.specvlm_argmax(lg, tok2)
    sv.specvlm_accept_compact(drf, par, tok2, k2, v2, pl, idx2, n2, nx2, nl2, st2)
    torch.cuda.synchronize()
    assert st1.item() == 0 and st2.item() == 0
    for a, b_ in ((k1, k2), (v1, v2), (tok1, tok2), (idx1, idx2), (n1, n2), (nx1, nx2), (nl1, nl2)):
        assert torch.equal(a, b_)
    assert n1.tolist() == [3, 4]
    # attention of both routes against the oracle on a few heads (the two routes may run different
    # kernel configurations, so they are compared through the oracle, not bitwise)
    for o in (o1, o2):
        for (l, b, h) in ((0, 0, 0), (3, 1, 7), (2, 0, 5)):
            ref = oracle.attention.tree_attn_bits(torch_to_bits(q[l, b, h]), torch_to_bits(k[l, b, h]),
                                                  torch_to_bits(v[l, b, h]), int(prefixes[b]),
                                                  oracle.tree_mask_bits(parents[b]))
            assert_attn_close(torch_to_bits(o[l, b, h]), ref)


def test_verify_step_sample_equals_per_call_sequence_and_oracle():
    """Temperature > 0: one call = attention per layer + accept_sample + kv_compact, and the
    acceptance and the compacted caches equal the oracle's on uniforms that are far from every
    decision threshold."""
    rng = np.random.default_rng(12)
    L, B, H, T, V = 3, 3, 4, 60, 32000
    temperature = 0.8
    prefixes = np.array([500, 333, 64], dtype=np.int32)
    S_cap = 500 + T
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(6)
    bf = dict(dtype=torch.bfloat16, device=dev)
    k = torch.randn((L, B, H, S_cap, 128), generator=gen, **bf)
    v = torch.randn((L, B, H, S_cap, 128), generator=gen, **bf)
    q = torch.randn((L, B, H, T, 128), generator=gen, **bf)
    parents, drafts, logits, uas, uss = [], [], [], [], []
    for b in range(B):
        p = wl.eagle2_like_tree(rng, T, 6)
        d = wl.sibling_distinct_tokens(rng, p, V)
        lg, _ = wl.planted_logits(rng, p, d, V, plant_len=2 + 2 * b, bump=8.0)
        lg = (lg * 3.0).astype(np.float32)
        for _ in range(500):
            ua, us = rng.random(T, dtype=np.float32), rng.random(T, dtype=np.float32)
            if oracle.decision_margins(p, d, lg, ua, us, temperature) >= 2e-5:
                break
        else:
            raise AssertionError("could not draw robust uniforms")
        parents.append(p), drafts.append(d), logits.append(lg), uas.append(ua), uss.append(us)
    i32 = dict(dtype=torch.int32, device=dev)
    par, drf = torch.tensor(np.array(parents), **i32), torch.tensor(np.array(drafts), **i32)
    lg = torch.from_numpy(np.stack(logits)).to(dev)
    ua, us = torch.from_numpy(np.stack(uas)).to(dev), torch.from_numpy(np.stack(uss)).to(dev)
    pl = torch.tensor(prefixes, **i32)
    mask = torch.zeros((B, T), dtype=torch.int64, device=dev)
    sv.specvlm_tree_build(par, pl, mask)

    def fresh():
        return (k.clone(), v.clone(), torch.zeros_like(q), torch.zeros((B, T, 2), device=dev),
                torch.zeros((B, 8), **i32), torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros(B, **i32),
                torch.zeros(1, **i32))

    k1, v1, o1, rs1, idx1, n1, nx1, nl1, st1 = fresh()
    sv.specvlm_verify_step_sample(q, k1, v1, pl, par, mask, drf, lg, ua, us, temperature, o1, rs1, idx1, n1, nx1, nl1,
                                  status=st1)
    k2, v2, o2, rs2, idx2, n2, nx2, nl2, st2 = fresh()
    for l in range(L):
        sv.specvlm_tree_verify_attn(q[l], k2[l], v2[l], pl, par, mask, o2[l], status=st2)
    sv.specvlm_accept_sample(drf, par, lg, ua, us, temperature, idx2, n2, nx2, rs2, st2)
    sv.specvlm_kv_compact(k2, v2, pl, idx2, n2, nl2, st2)
    torch.cuda.synchronize()
    assert st1.item() == 0 and st2.item() == 0
    for a, b_ in ((k1, k2), (v1, v2), (o1, o2), (rs1, rs2), (idx1, idx2), (n1, n2), (nx1, nx2), (nl1, nl2)):
        assert torch.equal(a, b_)
    kb, vb = torch_to_bits(k), torch_to_bits(v)
    full_idx = np.full((B, 64), -1, dtype=np.int32)
    lens = []
    for b in range(B):
        path, n_acc, tok = oracle.accept_sample(parents[b], drafts[b], logits[b], uas[b], uss[b], temperature)
        assert n1[b].item() == n_acc and nx1[b].item() == tok and idx1[b, :n_acc + 1].tolist() == path
        full_idx[b, :len(path)] = path
        lens.append(n_acc)
    assert max(lens) >= 1
    ek, ev, new_len = oracle.kv_compact(kb, vb, prefixes, full_idx, lens)
    assert np.array_equal(torch_to_bits(k1), ek) and np.array_equal(torch_to_bits(v1), ev)
    assert nl1.tolist() == list(new_len)
