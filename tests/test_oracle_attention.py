"""Pins of the oracle's attention on compacted heads (Eq. 2 with the heads of the "Coupled Weight Matrix in MHA"
reformulation restricted to their kept indices) against things other than itself: softmax row sums, closed forms,
the library's attention and autograd on the special case of equal head widths, central finite differences, the
restricted-product and masked-full-model identities, and invariance under zero padding of a head's block."""
import numpy as np
import pytest
import torch

from oracle import oracle as O

RAGGED_QK = [20, 21, 25, 37]
RAGGED_VO = [26, 30, 64, 13]


def layout(widths, gap=0):
    off, o = [], 0
    for w in widths:
        off.append(o)
        o += w + gap
    return np.array(off, dtype=np.int32), np.array(widths, dtype=np.int32), o


def rand_qkv(T, nq, nv, seed=0, dtype=torch.float64):
    g = torch.Generator().manual_seed(seed)
    r = lambda n: torch.randn((T, n), generator=g, dtype=torch.float64).to(dtype)
    return r(nq), r(nq), r(nv)


@pytest.mark.parametrize("causal", [False, True])
def test_softmax_rows_sum_to_one_and_mask(causal):
    batch, seq = 2, 19
    qo, qw, nq = layout(RAGGED_QK)
    vo, vw, nv = layout(RAGGED_VO)
    Q, K, V = rand_qkv(batch * seq, nq, nv)
    r = O.attn_fwd(Q, K, V, batch, seq, qo, qw, vo, vw, 0.125, causal, want_p=True)
    P = r["P"]
    np.testing.assert_allclose(P.sum(axis=-1), 1.0, rtol=0, atol=1e-13)
    assert (P >= 0).all()
    if causal:
        iu = np.triu_indices(seq, k=1)
        assert (P[:, :, iu[0], iu[1]] == 0).all()
        assert (P[:, :, 0, 0] == 1).all()
    # lse is the log of the softmax denominator: P_ij = exp(S_ij - lse_i)
    S = np.einsum("tc,uc->tu", Q[:seq, qo[1]:qo[1] + qw[1]].numpy(), K[:seq, qo[1]:qo[1] + qw[1]].numpy()) * 0.125
    if causal:
        S = np.where(np.tril(np.ones((seq, seq), dtype=bool)), S, -np.inf)
    np.testing.assert_allclose(np.exp(S - r["lse"][1, :seq, None]), P[1, 0], rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_zero_queries_give_the_mean_of_the_values(causal):
    batch, seq = 1, 11
    qo, qw, nq = layout([5, 7])
    vo, vw, nv = layout([3, 9])
    _, K, V = rand_qkv(seq, nq, nv, seed=1)
    Q = torch.zeros((seq, nq), dtype=torch.float64)
    ctx = O.attn_fwd(Q, K, V, batch, seq, qo, qw, vo, vw, 1.0, causal)["Ctx"]
    Vn = V.numpy()
    for i in range(seq):
        ref = Vn[: i + 1].mean(axis=0) if causal else Vn.mean(axis=0)
        np.testing.assert_allclose(ctx[i], ref, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_equal_widths_reduce_to_the_library_attention_and_its_autograd(causal):
    """Heads of one width d stored side by side are what torch's attention takes as (batch, heads, seq, d)."""
    batch, seq, H, d = 2, 17, 3, 8
    off = np.arange(H, dtype=np.int32) * d
    w = np.full(H, d, dtype=np.int32)
    Q, K, V = rand_qkv(batch * seq, H * d, H * d, seed=2)
    g = torch.Generator().manual_seed(9)
    dC = torch.randn((batch * seq, H * d), generator=g, dtype=torch.float64)
    scale = 1.0 / np.sqrt(d)
    split = lambda t: t.reshape(batch, seq, H, d).permute(0, 2, 1, 3)
    q, k, v = (split(t).clone().requires_grad_(True) for t in (Q, K, V))
    out = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=causal, scale=scale)
    merged = out.permute(0, 2, 1, 3).reshape(batch * seq, H * d)
    ours = O.attn_fwd(Q, K, V, batch, seq, off, w, off, w, scale, causal)
    np.testing.assert_allclose(ours["Ctx"], merged.detach().numpy(), rtol=1e-11, atol=1e-13)
    (merged * dC).sum().backward()
    back = O.attn_bwd(Q, K, V, dC, batch, seq, off, w, off, w, scale, causal)
    merge = lambda t: t.permute(0, 2, 1, 3).reshape(batch * seq, H * d).numpy()
    np.testing.assert_allclose(back["dQ"], merge(q.grad), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(back["dK"], merge(k.grad), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(back["dV"], merge(v.grad), rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_matches_central_finite_differences_on_ragged_heads(causal):
    batch, seq = 2, 7
    qo, qw, nq = layout([3, 5, 2])
    vo, vw, nv = layout([4, 1, 6])
    Q, K, V = rand_qkv(batch * seq, nq, nv, seed=3)
    g = torch.Generator().manual_seed(4)
    dC = torch.randn((batch * seq, nv), generator=g, dtype=torch.float64)
    scale = 0.37
    loss = lambda q, k, v: float((O.attn_fwd(q, k, v, batch, seq, qo, qw, vo, vw, scale, causal)["Ctx"] * dC.numpy()).sum())
    back = O.attn_bwd(Q, K, V, dC, batch, seq, qo, qw, vo, vw, scale, causal)
    eps = 1e-6
    r = np.random.default_rng(0)
    for name, idx in (("dQ", 0), ("dK", 1), ("dV", 2)):
        base = [Q, K, V]
        for _ in range(12):
            t, c = int(r.integers(batch * seq)), int(r.integers(base[idx].shape[1]))
            plus = [x.clone() for x in base]; minus = [x.clone() for x in base]
            plus[idx][t, c] += eps; minus[idx][t, c] -= eps
            fd = (loss(*plus) - loss(*minus)) / (2 * eps)
            assert abs(fd - back[name][t, c]) <= 1e-7 * max(1.0, abs(fd)), (name, t, c, fd, back[name][t, c])


def test_restricted_product_and_masked_full_model_identities():
    """Attention on the compacted heads equals attention of the full model whose removed columns of W_Q, W_K, W_V
    are zeroed (with the architectural 1/sqrt(d_h)), restricted to the kept value columns; and the logits of a
    compacted head are the sum over its kept indices of q_j k_j^T."""
    batch, seq, H, d_h, d_m = 1, 13, 3, 8, 24
    g = torch.Generator().manual_seed(5)
    X = torch.randn((seq, d_m), generator=g, dtype=torch.float64)
    WQ, WK, WV = (torch.randn((d_m, H * d_h), generator=g, dtype=torch.float64) * 0.3 for _ in range(3))
    r = np.random.default_rng(6)
    kept_qk = [np.sort(r.choice(d_h, size=k, replace=False)) for k in (3, 8, 5)]
    kept_vo = [np.sort(r.choice(d_h, size=k, replace=False)) for k in (6, 2, 8)]
    cq = np.concatenate([kk + h * d_h for h, kk in enumerate(kept_qk)])
    cv = np.concatenate([kk + h * d_h for h, kk in enumerate(kept_vo)])
    scale = 1.0 / np.sqrt(d_h)
    Qc, Kc, Vc = X @ WQ[:, cq], X @ WK[:, cq], X @ WV[:, cv]
    qo, qw, _ = layout([len(k) for k in kept_qk])
    vo, vw, _ = layout([len(k) for k in kept_vo])
    comp = O.attn_fwd(Qc, Kc, Vc, batch, seq, qo, qw, vo, vw, scale, False, want_p=True)
    # masked full model: zero the removed columns, run full-width heads
    mq = torch.zeros(H * d_h, dtype=torch.float64); mq[cq] = 1
    mv = torch.zeros(H * d_h, dtype=torch.float64); mv[cv] = 1
    Qf, Kf, Vf = X @ (WQ * mq), X @ (WK * mq), X @ (WV * mv)
    fo = np.arange(H, dtype=np.int32) * d_h
    fw = np.full(H, d_h, dtype=np.int32)
    full = O.attn_fwd(Qf, Kf, Vf, batch, seq, fo, fw, fo, fw, scale, False, want_p=True)
    np.testing.assert_allclose(comp["P"], full["P"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(comp["Ctx"], full["Ctx"][:, cv], rtol=1e-12, atol=1e-15)
    removed = np.setdiff1d(np.arange(H * d_h), cv)
    assert (full["Ctx"][:, removed] == 0).all()
    # restricted product, head 0: logits = sum over kept j of (X w^Q_j)(X w^K_j)^T
    S0 = sum(np.outer((X @ WQ[:, j]).numpy(), (X @ WK[:, j]).numpy()) for j in cq[: len(kept_qk[0])]) * scale
    P0 = np.exp(S0 - S0.max(axis=1, keepdims=True)); P0 /= P0.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(comp["P"][0, 0], P0, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_zero_padded_head_blocks_change_nothing(causal):
    """Giving every head's block extra zero columns (the padded layout a kernel with 16-element granularity reads)
    leaves outputs and gradients of the real columns unchanged and yields zeros in the pad columns."""
    batch, seq = 2, 9
    qo, qw, nq = layout(RAGGED_QK)
    vo, vw, nv = layout(RAGGED_VO)
    Q, K, V = rand_qkv(batch * seq, nq, nv, seed=7)
    g = torch.Generator().manual_seed(8)
    dC = torch.randn((batch * seq, nv), generator=g, dtype=torch.float64)
    pad = lambda w: -(-w // 16) * 16
    qo2, qw2, nq2 = layout([pad(w) for w in RAGGED_QK])
    vo2, vw2, nv2 = layout([pad(w) for w in RAGGED_VO])

    def spread(t, off, w, off2, n2):
        o = torch.zeros((t.shape[0], n2), dtype=t.dtype)
        for h in range(len(w)):
            o[:, off2[h]: off2[h] + w[h]] = t[:, off[h]: off[h] + w[h]]
        return o

    Q2, K2 = spread(Q, qo, qw, qo2, nq2), spread(K, qo, qw, qo2, nq2)
    V2, dC2 = spread(V, vo, vw, vo2, nv2), spread(dC, vo, vw, vo2, nv2)
    a = O.attn_fwd(Q, K, V, batch, seq, qo, qw, vo, vw, 0.2, causal)
    b = O.attn_fwd(Q2, K2, V2, batch, seq, qo2, qw2, vo2, vw2, 0.2, causal)
    ga = O.attn_bwd(Q, K, V, dC, batch, seq, qo, qw, vo, vw, 0.2, causal)
    gb = O.attn_bwd(Q2, K2, V2, dC2, batch, seq, qo2, qw2, vo2, vw2, 0.2, causal)
    for x, y, off, w, off2, n2 in ((a["Ctx"], b["Ctx"], vo, vw, vo2, nv2), (ga["dQ"], gb["dQ"], qo, qw, qo2, nq2),
                                   (ga["dK"], gb["dK"], qo, qw, qo2, nq2), (ga["dV"], gb["dV"], vo, vw, vo2, nv2)):
        np.testing.assert_array_equal(spread(torch.from_numpy(x), off, w, off2, n2).numpy(), y)
    np.testing.assert_array_equal(a["lse"], b["lse"])


def test_keys_shifted_by_a_constant_vector_leave_the_softmax_unchanged():
    batch, seq = 1, 10
    qo, qw, nq = layout([6])
    vo, vw, nv = layout([4])
    Q, K, V = rand_qkv(seq, nq, nv, seed=10)
    c = torch.randn((1, nq), generator=torch.Generator().manual_seed(11), dtype=torch.float64)
    a = O.attn_fwd(Q, K, V, batch, seq, qo, qw, vo, vw, 0.5, False)["Ctx"]
    b = O.attn_fwd(Q, K + c, V, batch, seq, qo, qw, vo, vw, 0.5, False)["Ctx"]
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-13)


def test_bf16_inputs_are_widened_exactly():
    batch, seq = 1, 6
    qo, qw, nq = layout([4, 4])
    vo, vw, nv = layout([4, 4])
    Q, K, V = rand_qkv(seq, nq, nv, seed=12, dtype=torch.bfloat16)
    a = O.attn_fwd(Q, K, V, batch, seq, qo, qw, vo, vw, 0.5, True)["Ctx"]
    b = O.attn_fwd(Q.double(), K.double(), V.double(), batch, seq, qo, qw, vo, vw, 0.5, True)["Ctx"]
    np.testing.assert_array_equal(a, b)


def test_compaction_with_pad_entries_inserts_zero_columns_and_rows():
    """A kept list with -1 entries (used to pad every head's block) gives zero columns / rows there and the plain
    gather elsewhere; the product of the padded pair equals the product of the plain compacted pair."""
    g = torch.Generator().manual_seed(13)
    W1 = torch.randn((5, 12), generator=g).to(torch.bfloat16)
    W2 = torch.randn((12, 7), generator=g).to(torch.bfloat16)
    kept = np.array([1, 4, 9, 10], dtype=np.int32)
    padded = np.array([1, 4, -1, -1, 9, 10, -1, -1], dtype=np.int32)
    a1, a2 = O.compact(W1, O.SHARED_COLS, kept), O.compact(W2, O.SHARED_ROWS, kept)
    b1, b2 = O.compact(W1, O.SHARED_COLS, padded), O.compact(W2, O.SHARED_ROWS, padded)
    real = padded >= 0
    assert torch.equal(b1[:, real], a1) and torch.equal(b2[real], a2)
    assert (b1[:, ~real] == 0).all() and (b2[~real] == 0).all()
    np.testing.assert_array_equal((b1.double() @ b2.double()).numpy(), (a1.double() @ a2.double()).numpy())
