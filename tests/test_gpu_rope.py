"""GPU parity: specvlm_rope_append (RoPE at tree positions + tree K/V append) against the oracle."""

import numpy as np
import pytest
import torch

import oracle
import paper_2509_11815_b200 as sv
import workloads as wl
from util import assert_attn_close, bits_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


def assert_rope_close(got_bits, x_f64, pos, base):
    """The kernel rotates in fp32 (angles reduced in double) and rounds once to bf16. Against the
    exact fp64 rotation that allows the bf16 rounding step (half an ulp = 2^-8 relative) plus the fp32 error of
    the two products, which is relative to |x_d| + |x_{d+64}|, not to a possibly cancelled result;
    and the result must be the correctly rounded one except for rare boundary cases."""
    exact = oracle.rope_rotate_half(x_f64, pos, base)
    got = oracle.bf16_bits_to_f64(got_bits)
    mag = np.abs(x_f64[..., :64]) + np.abs(x_f64[..., 64:])
    mag = np.concatenate([mag, mag], axis=-1)
    tol = 2.0 ** -8 * np.abs(exact) * 1.001 + 4e-6 * mag + 1e-30
    assert (np.abs(got - exact) <= tol).all(), float((np.abs(got - exact) - tol).max())
    differ = got_bits != oracle.f64_to_bf16_bits(exact)
    assert differ.sum() <= max(2, 2e-3 * differ.size), f"{differ.sum()} of {differ.size} elements are not correctly rounded"


def run_case(seed, B, H, T, prefixes, tree_kind="eagle", base=0.0, in_place=False):
    rng = np.random.default_rng(seed)
    S_cap = int(max(prefixes)) + T + 3
    parents = []
    for b in range(B):
        if tree_kind == "chain":
            parents.append(wl.chain_tree(T))
        elif T >= 20:
            parents.append(wl.eagle2_like_tree(rng, T, min(6, T - 1)))
        else:
            parents.append(wl.config1_tree(rng, T, min(4, T - 1)) if T > 1 else wl.single_node_tree())
    parents = np.array(parents, dtype=np.int32)
    q = wl.normal_bf16_bits(rng, (B, H, T, 128))
    kn = wl.normal_bf16_bits(rng, (B, H, T, 128))
    vn = wl.normal_bf16_bits(rng, (B, H, T, 128))
    kc = wl.normal_bf16_bits(rng, (B, H, S_cap, 128))
    vc = wl.normal_bf16_bits(rng, (B, H, S_cap, 128))
    tq, tkn, tvn, tkc, tvc = (bits_to_torch(x) for x in (q, kn, vn, kc, vc))
    q_out = tq if in_place else torch.zeros_like(tq)
    i32 = dict(dtype=torch.int32, device="cuda")
    pl = torch.tensor(np.asarray(prefixes), **i32)
    pos = torch.full((B, T), -7, **i32)
    status = torch.zeros(1, **i32)
    sv.specvlm_rope_append(tq, tkn, tvn, pl, torch.tensor(parents, **i32), q_out, tkc, tvc, pos, status, base)
    torch.cuda.synchronize()
    assert status.item() == 0
    rope_base = base if base > 0 else 10000.0
    exp_kc, exp_vc = kc.copy(), vc.copy()
    got_kc, got_vc, got_q = torch_to_bits(tkc), torch_to_bits(tvc), torch_to_bits(q_out)
    for b in range(B):
        P = int(prefixes[b])
        p_ids = oracle.tree_positions(parents[b], P)
        assert np.array_equal(pos[b].cpu().numpy(), p_ids)
        for h in range(H):
            assert_rope_close(got_q[b, h], oracle.bf16_bits_to_f64(q[b, h]), p_ids, rope_base)
            assert_rope_close(got_kc[b, h, P:P + T], oracle.bf16_bits_to_f64(kn[b, h]), p_ids, rope_base)
        exp_vc[b, :, P:P + T] = vn[b]
        exp_kc[b, :, P:P + T] = got_kc[b, :, P:P + T]   # checked above; the rest must be untouched
    assert np.array_equal(got_vc, exp_vc) and np.array_equal(got_kc, exp_kc)
    return parents, q, got_q, got_kc, got_vc


@pytest.mark.parametrize("T", [1, 7, 26, 60, 64])
def test_rope_append_matches_oracle(T):
    run_case(T, B=3, H=5, T=T, prefixes=[0, 333, 9728])


@pytest.mark.parametrize("B,H", [(1, 32), (2, 40), (70, 9)])
def test_rope_append_head_distribution_over_blocks(B, H):
    """One head per warp (H a multiple of the warps per block or not), and a batch large enough
    that a warp loops over several heads."""
    rng = np.random.default_rng(B * H)
    run_case(B * 100 + H, B=B, H=H, T=60, prefixes=rng.integers(0, 120, size=B).tolist())


def test_rope_append_in_place_custom_base_and_strided_cache():
    run_case(99, B=2, H=4, T=60, prefixes=[3008, 17], base=500000.0, in_place=True)


def test_rope_append_bad_inputs_set_status_and_skip():
    rng = np.random.default_rng(5)
    B, H, T = 2, 2, 6
    tq = bits_to_torch(wl.normal_bf16_bits(rng, (B, H, T, 128)))
    kc = wl.normal_bf16_bits(rng, (B, H, 40, 128))
    tkc, tvc = bits_to_torch(kc), bits_to_torch(kc)
    i32 = dict(dtype=torch.int32, device="cuda")
    parents = torch.tensor([[-1, 0, 0, 1, 1, 2], [-1, 0, 3, 1, 1, 2]], **i32)     # second tree malformed
    status = torch.zeros(1, **i32)
    q_out = torch.zeros_like(tq)
    sv.specvlm_rope_append(tq, tq, tq, torch.tensor([10, 10], **i32), parents, q_out, tkc, tvc, None, status)
    torch.cuda.synchronize()
    assert status.item() & sv.STATUS_BAD_TREE
    got = torch_to_bits(tkc)
    assert not np.array_equal(got[0], kc[0])
    status.zero_()
    sv.specvlm_rope_append(tq, tq, tq, torch.tensor([10, 36], **i32), parents[:1].repeat(2, 1), q_out, tkc, tvc,
                           None, status)
    torch.cuda.synchronize()
    assert status.item() & sv.STATUS_BAD_PREFIX


def test_rope_append_then_attention_on_a_chain_is_causal_attention():
    """End to end on the GPU: rotate + append the chain's rows, then tree attention; the result
    is ordinary causal attention over P + T tokens at positions 0..P+T-1."""
    rng = np.random.default_rng(6)
    H, T, P = 2, 24, 150
    n = P + T
    q_all = wl.normal_bf16_bits(rng, (1, H, n, 128))
    k_all = wl.normal_bf16_bits(rng, (1, H, n, 128))
    v_all = wl.normal_bf16_bits(rng, (1, H, n, 128))
    qf, kf, vf = (oracle.bf16_bits_to_f64(x) for x in (q_all, k_all, v_all))
    kc = np.zeros((1, H, n, 128), dtype=np.uint16)
    for h in range(H):   # the prefix was rotated when it was generated
        kc[0, h, :P] = oracle.f64_to_bf16_bits(oracle.rope_rotate_half(kf[0, h, :P], np.arange(P)))
    vc = v_all.copy()
    vc[0, :, P:] = 0
    tkc, tvc = bits_to_torch(kc), bits_to_torch(vc)
    i32 = dict(dtype=torch.int32, device="cuda")
    par = torch.tensor(wl.chain_tree(T)[None], **i32)
    pl = torch.tensor([P], **i32)
    tq = bits_to_torch(np.ascontiguousarray(q_all[:, :, P:]))
    q_rot = torch.zeros_like(tq)
    sv.specvlm_rope_append(tq, bits_to_torch(np.ascontiguousarray(k_all[:, :, P:])),
                           bits_to_torch(np.ascontiguousarray(v_all[:, :, P:])), pl, par, q_rot, tkc, tvc)
    out = torch.zeros_like(tq)
    sv.specvlm_tree_verify_attn(q_rot, tkc, tvc, pl, par, None, out)
    torch.cuda.synchronize()
    # reference: rotate in fp64, round q/k to bf16 as the kernels do, then textbook causal attention
    for h in range(H):
        pos = np.arange(n)
        qr = oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(oracle.rope_rotate_half(qf[0, h], pos)))
        kr = oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(oracle.rope_rotate_half(kf[0, h], pos)))
        causal = oracle.causal_attn_textbook(qr, kr, vf[0, h])[P:]
        assert_attn_close(torch_to_bits(out)[0, h], causal)
