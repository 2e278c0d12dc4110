"""Pins of the oracle's attention core for grouped-query models (Sec. 3.1, "Extension to GQA").

(1) With one query head per K/V head it is the multi-head routine.  (2) Against the library's grouped attention
(`scaled_dot_product_attention` on K/V repeated per query head, fp64) and its autograd, which adds the gradients of the
repeated heads: outputs, dQ, dK, dV.  (3) A group whose query heads are identical gives every head of the group the same
output, and dK, dV equal to the group size times one head's contribution.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O


def layout(widths):
    off, o = [], 0
    for w in widths:
        off.append(o)
        o += w
    return off, o


def make(batch, seq, wq_g, wv_g, rep, seed=0):
    g = torch.Generator().manual_seed(seed)
    G = len(wq_g)
    qk_w = [wq_g[h // rep] for h in range(G * rep)]
    vo_w = [wv_g[h // rep] for h in range(G * rep)]
    qk_off, n_q = layout(qk_w)
    vo_off, n_vo = layout(vo_w)
    k_off, n_k = layout(wq_g)
    v_off, n_v = layout(wv_g)
    T = batch * seq
    r = lambda n: torch.randn((T, n), generator=g, dtype=torch.float64)
    return dict(Q=r(n_q), K=r(n_k), V=r(n_v), dCtx=r(n_vo), qk_off=qk_off, qk_w=qk_w, vo_off=vo_off, vo_w=vo_w, k_off=k_off,
                v_off=v_off)


@pytest.mark.parametrize("causal", [False, True])
def test_one_query_head_per_kv_head_is_multi_head_attention(causal):
    d = make(2, 19, [5, 8, 3], [4, 2, 7], 1, seed=1)
    a = O.attn_fwd_gqa(d["Q"], d["K"], d["V"], 2, 19, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], 0.3, causal)
    b = O.attn_fwd(d["Q"], d["K"], d["V"], 2, 19, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], 0.3, causal)
    assert np.array_equal(a["Ctx"], b["Ctx"]) and np.array_equal(a["lse"], b["lse"])
    ga = O.attn_bwd_gqa(d["Q"], d["K"], d["V"], d["dCtx"], 2, 19, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], 0.3, causal)
    gb = O.attn_bwd(d["Q"], d["K"], d["V"], d["dCtx"], 2, 19, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], 0.3, causal)
    for k in ("dQ", "dK", "dV"):
        assert np.array_equal(ga[k], gb[k])


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("rep", [2, 4])
def test_against_the_library_attention_on_repeated_heads_and_its_autograd(rep, causal):
    batch, seq, w, G = 2, 23, 6, 3
    d = make(batch, seq, [w] * G, [w] * G, rep, seed=rep)
    H = G * rep
    scale = 0.37
    Q = d["Q"].clone().requires_grad_(True)
    K = d["K"].clone().requires_grad_(True)
    V = d["V"].clone().requires_grad_(True)
    q4 = Q.view(batch, seq, H, w).transpose(1, 2)
    k4 = K.view(batch, seq, G, w).transpose(1, 2).repeat_interleave(rep, dim=1)
    v4 = V.view(batch, seq, G, w).transpose(1, 2).repeat_interleave(rep, dim=1)
    out = torch.nn.functional.scaled_dot_product_attention(q4, k4, v4, is_causal=causal, scale=scale)
    ctx = out.transpose(1, 2).reshape(batch * seq, H * w)
    ctx.backward(d["dCtx"])
    a = O.attn_fwd_gqa(d["Q"], d["K"], d["V"], batch, seq, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], scale, causal)
    np.testing.assert_allclose(a["Ctx"], ctx.detach().numpy(), rtol=1e-10, atol=1e-12)
    g = O.attn_bwd_gqa(d["Q"], d["K"], d["V"], d["dCtx"], batch, seq, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], scale, causal)
    np.testing.assert_allclose(g["dQ"], Q.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(g["dK"], K.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(g["dV"], V.grad.numpy(), rtol=1e-9, atol=1e-11)


def test_identical_query_heads_of_a_group():
    batch, seq, rep = 1, 17, 3
    d = make(batch, seq, [4, 7], [5, 3], rep, seed=9)
    for g in range(2):                                     # every head of a group gets the group's first head's queries
        for r in range(1, rep):
            h0, h = g * rep, g * rep + r
            d["Q"][:, d["qk_off"][h]: d["qk_off"][h] + d["qk_w"][h]] = d["Q"][:, d["qk_off"][h0]: d["qk_off"][h0] + d["qk_w"][h0]]
            d["dCtx"][:, d["vo_off"][h]: d["vo_off"][h] + d["vo_w"][h]] = d["dCtx"][:, d["vo_off"][h0]: d["vo_off"][h0] + d["vo_w"][h0]]
    a = O.attn_fwd_gqa(d["Q"], d["K"], d["V"], batch, seq, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], 0.5, True)
    gq = O.attn_bwd_gqa(d["Q"], d["K"], d["V"], d["dCtx"], batch, seq, d["qk_off"], d["qk_w"], d["vo_off"], d["vo_w"], d["k_off"], d["v_off"], 0.5, True)
    # one head per group on its own
    one = dict(qk_off=[d["qk_off"][0], d["qk_off"][rep]], qk_w=[d["qk_w"][0], d["qk_w"][rep]], vo_off=[d["vo_off"][0], d["vo_off"][rep]],
               vo_w=[d["vo_w"][0], d["vo_w"][rep]])
    g1 = O.attn_bwd_gqa(d["Q"], d["K"], d["V"], d["dCtx"], batch, seq, one["qk_off"], one["qk_w"], one["vo_off"], one["vo_w"], d["k_off"], d["v_off"], 0.5, True)
    for g in range(2):
        for r in range(1, rep):
            h0, h = g * rep, g * rep + r
            assert np.array_equal(a["Ctx"][:, d["vo_off"][h]: d["vo_off"][h] + d["vo_w"][h]], a["Ctx"][:, d["vo_off"][h0]: d["vo_off"][h0] + d["vo_w"][h0]])
    np.testing.assert_allclose(gq["dK"], rep * g1["dK"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(gq["dV"], rep * g1["dV"], rtol=1e-12, atol=1e-14)
