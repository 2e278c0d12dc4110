"""Pins of the grouped-query reading: the query heads that share a K/V head share its kept index set, and the group
is scored as one coupled pair whose shared side is the stack of the group's heads ("Extension to GQA": the coupled
matrices W_i^Q W_g(i)^K^T and W_g(i)^V W_i^O).  Pinned by: the plain pair score of the explicitly stacked matrices,
the reduction to ordinary heads when every group has one head, Proposition 1 over the group by brute force, and the
restricted-product identity per query head."""
import numpy as np
import torch

from oracle import oracle as O


def rand(shape, seed):
    return torch.randn(shape, generator=torch.Generator().manual_seed(seed), dtype=torch.float64)


def test_group_score_is_the_plain_score_of_the_stacked_pair():
    d_m, d_h, n_groups, rep = 12, 6, 3, 4
    WQ = rand((d_m, n_groups * rep * d_h), 0)          # query heads side by side, a group's heads adjacent
    WK = rand((d_m, n_groups * d_h), 1)
    raw, ups = O.score_pair_gqa(WQ, WK, O.SHARED_COLS, O.SHARED_COLS, n_groups, d_h, rep1=rep)
    for g in range(n_groups):
        heads = [WQ[:, (g * rep + r) * d_h:(g * rep + r + 1) * d_h] for r in range(rep)]
        stack = torch.cat(heads, dim=0).contiguous()       # (rep * d_m) x d_h: W_1 of the group's coupled pair
        wk = WK[:, g * d_h:(g + 1) * d_h].contiguous()
        raw_s, ups_s = O.score_pair(stack, wk, O.SHARED_COLS, O.SHARED_COLS, 1, d_h)
        np.testing.assert_allclose(raw[g * d_h:(g + 1) * d_h], raw_s, rtol=1e-13)
        np.testing.assert_allclose(ups[g * d_h:(g + 1) * d_h], ups_s, rtol=1e-13)
    # V/O side: the group's W^O row blocks side by side are W_2 of the pair
    WV = rand((d_m, n_groups * d_h), 2)
    WO = rand((n_groups * rep * d_h, d_m), 3)
    raw, ups = O.score_pair_gqa(WV, WO, O.SHARED_COLS, O.SHARED_ROWS, n_groups, d_h, rep2=rep)
    for g in range(n_groups):
        blocks = [WO[(g * rep + r) * d_h:(g * rep + r + 1) * d_h] for r in range(rep)]
        wide = torch.cat(blocks, dim=1).contiguous()       # d_h x (rep * d_m)
        wv = WV[:, g * d_h:(g + 1) * d_h].contiguous()
        raw_s, _ = O.score_pair(wv, wide, O.SHARED_COLS, O.SHARED_ROWS, 1, d_h)
        np.testing.assert_allclose(raw[g * d_h:(g + 1) * d_h], raw_s, rtol=1e-13)


def test_groups_of_one_head_are_ordinary_heads():
    WQ, WK = rand((8, 20), 4), rand((8, 20), 5)
    a = O.score_pair_gqa(WQ, WK, 0, 0, 4, 5, rep1=1)
    b = O.score_pair(WQ, WK, 0, 0, 4, 5)
    np.testing.assert_array_equal(a[0], b[0]); np.testing.assert_array_equal(a[1], b[1])
    GQ, GK = rand((8, 20), 6), rand((8, 20), 7)
    np.testing.assert_allclose(O.fisher_pair_gqa(GQ, GK, 0, 0, 4, 5, 3.0), O.fisher_pair(GQ, GK, 0, 0, 4, 5, 3.0), rtol=1e-13)


def test_removing_the_lowest_scored_index_minimises_the_error_over_the_group():
    """Proposition 1 for the group: dropping index j from every pair of the group costs
    sqrt(sum_i ||W_i^Q W_g^K^T - (W_i^Q)_{-j} (W_g^K)_{-j}^T||_F^2) = raw[j], minimised by the lowest score."""
    d_m, d_h, rep = 7, 5, 3
    WQ, WK = rand((d_m, rep * d_h), 8), rand((d_m, d_h), 9)
    raw, _ = O.score_pair_gqa(WQ, WK, 0, 0, 1, d_h, rep1=rep)
    errs = []
    for j in range(d_h):
        keep = [c for c in range(d_h) if c != j]
        e2 = 0.0
        for r in range(rep):
            q = WQ[:, r * d_h:(r + 1) * d_h]
            e2 += float(((q @ WK.T) - (q[:, keep] @ WK[:, keep].T)).pow(2).sum())
        errs.append(np.sqrt(e2))
    np.testing.assert_allclose(errs, raw, rtol=1e-12)
    assert int(np.argmin(errs)) == int(np.argmin(raw))


def test_restricted_product_per_query_head():
    d_m, d_h, rep = 6, 8, 2
    WQ, WK = rand((d_m, rep * d_h), 10), rand((d_m, d_h), 11)
    _, ups = O.score_pair_gqa(WQ, WK, 0, 0, 1, d_h, rep1=rep)
    kept = O.select_topk(ups, 1, d_h, [5])
    assert len(kept) == 5
    kc = O.compact(WK, O.SHARED_COLS, kept)
    for r in range(rep):
        kept_q = kept + r * d_h                        # the same indices inside every query head of the group
        qc = O.compact(WQ, O.SHARED_COLS, kept_q)
        ref = sum(torch.outer(WQ[:, r * d_h + j], WK[:, j]) for j in kept)
        np.testing.assert_allclose((qc @ kc.T).numpy(), ref.numpy(), rtol=1e-12, atol=1e-14)


def test_constant_gradients_closed_form():
    n_groups, rep, d_h, d_m = 2, 3, 4, 5
    GQ = torch.full((d_m, n_groups * rep * d_h), 0.5, dtype=torch.float64)
    GK = torch.full((d_m, n_groups * d_h), 2.0, dtype=torch.float64)
    f = O.fisher_pair_gqa(GQ, GK, 0, 0, n_groups, d_h, 10.0, rep1=rep)
    np.testing.assert_allclose(f, 0.5 * (0.25 + 4.0) / 10.0, rtol=1e-14)
