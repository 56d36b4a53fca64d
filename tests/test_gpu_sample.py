"""GPU parity: specvlm_accept_sample (temperature > 0 tree acceptance) against the oracle."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl

pytestmark = pytest.mark.gpu


def gpu_accept_sample(parents, drafts, logits, ua, us, temperature, acc_stride=8):
    i32 = dict(dtype=torch.int32, device="cuda")
    B, T = parents.shape
    idx = torch.full((B, acc_stride), -99, **i32)
    n, nxt = torch.full((B,), -99, **i32), torch.full((B,), -99, **i32)
    status = torch.zeros(1, **i32)
    stats = torch.full((B, T, 2), float("nan"), dtype=torch.float32, device="cuda")
    sv.specvlm_accept_sample(torch.tensor(drafts, **i32), torch.tensor(parents, **i32),
                             torch.from_numpy(np.ascontiguousarray(logits, dtype=np.float32)).cuda(),
                             torch.from_numpy(np.ascontiguousarray(ua, dtype=np.float32)).cuda(),
                             torch.from_numpy(np.ascontiguousarray(us, dtype=np.float32)).cuda(),
                             temperature, idx, n, nxt, stats, status)
    torch.cuda.synchronize()
    # the row statistics are an output too: max bit-exact, partition sum = 1 / (largest probability)
    lg64 = np.asarray(logits, dtype=np.float64)
    got = stats.cpu().numpy()
    for b in range(min(B, 16)):
        for t in range(0, T, 7):
            p = oracle.softmax_f64(lg64[b, t], temperature)
            assert got[b, t, 0] == np.float32(lg64[b, t].max())
            assert abs(got[b, t, 1] * p.max() - 1.0) < 2e-5, (b, t, got[b, t, 1], 1.0 / p.max())
    return idx.cpu().numpy(), n.cpu().numpy(), nxt.cpu().numpy(), status.item()


def draw_robust_uniforms(rng, parent, draft, logits, temperature, margin):
    """float32 uniforms whose decisions all lie at least `margin` away from their thresholds, so
    that an fp32 evaluation must take the same decisions as the fp64 oracle."""
    for _ in range(500):
        ua = rng.random(len(parent), dtype=np.float32)
        us = rng.random(len(parent), dtype=np.float32)
        if oracle.decision_margins(parent, draft, logits, ua, us, temperature) >= margin:
            return ua, us
    raise AssertionError("could not draw robust uniforms")


@pytest.mark.parametrize("V,temperature,scale", [(32000, 1.0, 3.0), (32000, 0.7, 2.0), (1000, 1.0, 1.0), (17, 1.3, 1.0), (40000, 1.0, 3.0),
                                                 (32768, 0.8, 2.0), (1026, 1.0, 2.0)])
def test_accept_sample_matches_oracle_on_robust_draws(V, temperature, scale):
    rng = np.random.default_rng(V)
    B, T = 12, 60
    parents, drafts, logits, uas, uss = [], [], [], [], []
    for b in range(B):
        p = wl.eagle2_like_tree(rng, T, 6)
        d = wl.sibling_distinct_tokens(rng, p, V)
        lg, _ = wl.planted_logits(rng, p, d, V, plant_len=int(rng.integers(0, 7)), bump=8.0)
        lg = (lg * scale).astype(np.float32)
        ua, us = draw_robust_uniforms(rng, p, d, lg, temperature, margin=2e-5)
        parents.append(p), drafts.append(d), logits.append(lg), uas.append(ua), uss.append(us)
    parents, drafts = np.array(parents, dtype=np.int32), np.array(drafts, dtype=np.int32)
    idx, n, nxt, status = gpu_accept_sample(parents, drafts, np.stack(logits), np.stack(uas), np.stack(uss), temperature)
    assert status == 0
    lens = []
    for b in range(B):
        path, k, tok = oracle.accept_sample(parents[b], drafts[b], logits[b], uas[b], uss[b], temperature)
        lens.append(k)
        assert n[b] == k and nxt[b] == tok, (b, n[b], k, nxt[b], tok)
        want = np.full(8, -1)
        want[:min(8, len(path))] = path[:8]
        assert idx[b].tolist() == want.tolist()
    assert max(lens) >= 1


def test_kernel_output_follows_the_target_distribution():
    """Losslessness of the kernel itself: over many sequences with independent uniforms the first
    emitted token is distributed as softmax(logits_root / temperature)."""
    rng = np.random.default_rng(3)
    V, B, T = 8, 40000, 6
    parent = np.array([-1, 0, 0, 0, 1, 1], dtype=np.int32)
    draft = np.array([0, 4, 1, 5, 2, 3], dtype=np.int32)
    row = rng.standard_normal((T, V)).astype(np.float32)
    temperature = 0.9
    idx, n, nxt, status = gpu_accept_sample(np.tile(parent, (B, 1)), np.tile(draft, (B, 1)), np.tile(row, (B, 1, 1)),
                                            rng.random((B, T), dtype=np.float32), rng.random((B, T), dtype=np.float32),
                                            temperature, acc_stride=4)
    assert status == 0
    first = np.where(n >= 1, draft[np.maximum(idx[:, 1], 0)], nxt)
    counts = np.bincount(first, minlength=V).astype(np.float64)
    p = oracle.softmax_f64(row[0], temperature)
    chi2 = ((counts - B * p) ** 2 / (B * p)).sum()
    assert chi2 < 30.0, chi2                          # 7 degrees of freedom: P(chi2 > 30) ~ 1e-4
    sel = (n >= 1) & (idx[:, 1] == 1)                  # second token given that child 1 was kept
    second = np.where(n[sel] >= 2, draft[np.maximum(idx[sel, 2], 0)], nxt[sel])
    c2 = np.bincount(second, minlength=V).astype(np.float64)
    p1 = oracle.softmax_f64(row[1], temperature)
    chi2 = ((c2 - sel.sum() * p1) ** 2 / (sel.sum() * p1)).sum()
    assert chi2 < 30.0, chi2


def test_accept_sample_low_temperature_equals_greedy_kernel_and_rejects_bad_input():
    rng = np.random.default_rng(4)
    B, T, V = 6, 26, 500
    parents = np.array([wl.config1_tree(rng, T, 5) for _ in range(B)], dtype=np.int32)
    drafts = np.array([wl.sibling_distinct_tokens(rng, p, V) for p in parents], dtype=np.int32)
    logits = np.stack([wl.planted_logits(rng, parents[b], drafts[b], V, plant_len=b % 5)[0] for b in range(B)])
    ua, us = rng.random((B, T), dtype=np.float32) * 0.98 + 0.01, rng.random((B, T), dtype=np.float32) * 0.98 + 0.01
    idx, n, nxt, status = gpu_accept_sample(parents, drafts, logits, ua, us, temperature=0.01)
    assert status == 0
    for b in range(B):
        path, k, tok = oracle.accept_topdown(parents[b], drafts[b], oracle.vocab_argmax(logits[b]))
        assert n[b] == k and nxt[b] == tok and idx[b, :k + 1].tolist() == path
    with pytest.raises(sv.SpecvlmError):
        gpu_accept_sample(parents, drafts, logits, ua, us, temperature=0.0)
