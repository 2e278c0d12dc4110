"""Pins for the oracle's score / Fisher / selection / compaction functions.

Every check here compares the oracle with something it does not compute itself:
closed forms, invariances the definitions imply, brute force over tiny inputs, a
library routine on a special case, or numbers the paper prints.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
COLS, ROWS = O.SHARED_COLS, O.SHARED_ROWS


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------------------
# sum of squares / upsilon  (Eq. "l2norm")
# ---------------------------------------------------------------------------

def test_sumsq_closed_form_columns_and_rows():
    m, d, p = 5, 7, 3
    W1 = np.zeros((m, d))
    for j in range(d):
        W1[j % m, j] = j + 1.0           # column j has a single entry j+1  -> squared norm (j+1)^2
    v = np.array([0.5, 2.0, 1.0, 3.0, 0.25, 4.0, 1.5])
    W2 = np.repeat(v[:, None], p, axis=1)  # row j constant v_j  -> squared norm p v_j^2
    c1 = O.sumsq_shared(W1, COLS)
    c2 = O.sumsq_shared(W2, ROWS)
    np.testing.assert_allclose(c1, (np.arange(d) + 1.0) ** 2, rtol=0, atol=0)
    np.testing.assert_allclose(c2, p * v ** 2, rtol=1e-15)
    raw, ups = O.upsilon(c1, c2, 1, d)
    expect = (np.arange(d) + 1.0) * np.sqrt(p) * v
    np.testing.assert_allclose(raw, expect, rtol=1e-14)
    np.testing.assert_allclose(ups, expect / np.sqrt((expect ** 2).sum()), rtol=1e-14)


def test_sumsq_is_not_transposed():
    # a non-square matrix whose row sums and column sums differ: catches a swapped axis
    W = np.arange(1.0, 13.0).reshape(3, 4)
    np.testing.assert_allclose(O.sumsq_shared(W, COLS), (W ** 2).sum(0))
    np.testing.assert_allclose(O.sumsq_shared(W, ROWS), (W ** 2).sum(1))
    # the same matrix stored the other way round gives the same per-index numbers
    np.testing.assert_allclose(O.sumsq_shared(np.ascontiguousarray(W.T), ROWS), (W ** 2).sum(0))


def test_sumsq_dtypes_agree():
    t = torch.randn(33, 50, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    a = O.sumsq_shared(t, COLS)
    b = O.sumsq_shared(t.double(), COLS)
    c = O.sumsq_shared(t.float(), COLS)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(a, c)


def test_hadamard_reduces_to_plain_when_one_factor_is_ones():
    r = rng(2)
    W = r.standard_normal((9, 11))
    np.testing.assert_allclose(O.sumsq_shared_hadamard(np.ones_like(W), W, COLS), O.sumsq_shared(W, COLS), rtol=1e-15)
    np.testing.assert_allclose(O.sumsq_shared_hadamard(W, np.ones_like(W), COLS), O.sumsq_shared(W, COLS), rtol=1e-15)
    # element-wise product, not product of norms: a column where gate and up never overlap scores zero
    g = np.zeros((4, 2)); u = np.zeros((4, 2))
    g[0, 0] = 3.0; u[1, 0] = 5.0          # disjoint support -> (g.u) column is zero
    g[2, 1] = 2.0; u[2, 1] = 7.0          # overlapping -> 14^2
    np.testing.assert_allclose(O.sumsq_shared_hadamard(g, u, COLS), [0.0, 196.0])


def test_upsilon_unit_norm_per_segment_and_scale_invariance():
    r = rng(3)
    n_seg, seg_len, m, p = 3, 8, 6, 5
    D = n_seg * seg_len
    W1 = r.standard_normal((m, D)); W2 = r.standard_normal((D, p))
    raw, ups = O.score_pair(W1, W2, COLS, ROWS, n_seg, seg_len)
    for s in range(n_seg):
        seg = slice(s * seg_len, (s + 1) * seg_len)
        assert abs((ups[seg] ** 2).sum() - 1.0) < 1e-14
        np.testing.assert_allclose(ups[seg], raw[seg] / np.linalg.norm(raw[seg]), rtol=1e-14)
    _, ups2 = O.score_pair(3.5 * W1, 0.01 * W2, COLS, ROWS, n_seg, seg_len)
    np.testing.assert_allclose(ups2, ups, rtol=1e-12)
    # normalisation is per segment, not over the whole matrix
    assert abs((ups ** 2).sum() - n_seg) < 1e-13


def test_raw_invariant_under_balanced_rescaling():
    # scaling column j of W_1 by c and row j of W_2 by 1/c leaves W_1 W_2 and raw[j] unchanged
    r = rng(4)
    W1 = r.standard_normal((6, 10)); W2 = r.standard_normal((10, 4))
    c = r.uniform(0.2, 5.0, size=10)
    raw0, _ = O.score_pair(W1, W2, COLS, ROWS, 1, 10)
    raw1, _ = O.score_pair(W1 * c[None, :], W2 / c[:, None], COLS, ROWS, 1, 10)
    np.testing.assert_allclose(raw1, raw0, rtol=1e-13)
    np.testing.assert_allclose((W1 * c[None, :]) @ (W2 / c[:, None]), W1 @ W2, rtol=1e-12, atol=1e-12)


def test_permutation_equivariance():
    r = rng(5)
    d = 12
    W1 = r.standard_normal((7, d)); W2 = r.standard_normal((d, 5))
    perm = r.permutation(d)
    _, ups = O.score_pair(W1, W2, COLS, ROWS, 1, d)
    _, ups_p = O.score_pair(W1[:, perm], W2[perm, :], COLS, ROWS, 1, d)
    np.testing.assert_allclose(ups_p, ups[perm], rtol=1e-13)
    kept = set(O.select_topk(ups, 1, d, [5]).tolist())
    kept_p = set(perm[O.select_topk(ups_p, 1, d, [5])].tolist())
    assert kept == kept_p


def test_zero_segment_gives_zero_scores_and_first_k():
    W1 = np.zeros((4, 6)); W2 = np.ones((6, 3))
    W1[:, 3:] = 1.0                        # segment 0 is dead, segment 1 alive
    raw, ups = O.score_pair(W1, W2, COLS, ROWS, 2, 3)
    assert np.all(ups[:3] == 0.0) and np.all(np.isfinite(ups))
    kept = O.select_topk(ups, 2, 3, [2, 1])
    assert kept.tolist() == [0, 1, 3]


# ---------------------------------------------------------------------------
# Fisher importance (Eq. "importance")
# ---------------------------------------------------------------------------

def test_fisher_constant_gradients_closed_form():
    n_seg, seg_len, m, p, n_samples = 3, 4, 5, 7, 64.0
    D = n_seg * seg_len
    c1 = np.array([0.5, 2.0, 3.0]); c2 = np.array([1.0, 0.1, 4.0])
    G1 = np.repeat(c1, seg_len)[None, :] * np.ones((m, D))
    G2 = np.repeat(c2, seg_len)[:, None] * np.ones((D, p))
    f = O.fisher_pair(G1, G2, COLS, ROWS, n_seg, seg_len, n_samples)
    np.testing.assert_allclose(f, 0.5 * (c1 ** 2 + c2 ** 2) / n_samples, rtol=1e-14)
    # equal constants: I_hat = c^2 / n_samples whatever the two matrices' sizes
    f1 = O.fisher_pair(0.3 * np.ones((m, D)), 0.3 * np.ones((D, p)), COLS, ROWS, n_seg, seg_len, n_samples)
    np.testing.assert_allclose(f1, 0.09 / n_samples, rtol=1e-14)


def test_fisher_swiglu_slot_is_mean_of_gate_and_up():
    n_seg, seg_len, m, p = 1, 6, 4, 3
    Gg = 2.0 * np.ones((m, seg_len)); Gu = 4.0 * np.ones((m, seg_len)); Gd = 1.0 * np.ones((seg_len, p))
    f = O.fisher_pair(Gg, Gd, COLS, ROWS, n_seg, seg_len, 10.0, g1b=Gu)
    np.testing.assert_allclose(f, [0.5 * (0.5 * (4.0 + 16.0) + 1.0) / 10.0], rtol=1e-14)


def test_fisher_matches_library_sum_on_random_blocks():
    r = rng(7)
    n_seg, seg_len, m, p = 2, 5, 6, 4
    D = n_seg * seg_len
    G1 = r.standard_normal((m, D)); G2 = r.standard_normal((D, p))
    f = O.fisher_pair(G1, G2, COLS, ROWS, n_seg, seg_len, 3.0)
    for s in range(n_seg):
        seg = slice(s * seg_len, (s + 1) * seg_len)
        e = 0.5 * (np.mean(G1[:, seg] ** 2) + np.mean(G2[seg, :] ** 2)) / 3.0
        assert abs(f[s] - e) < 1e-14
    # layouts: the same gradients stored transposed give the same numbers
    f_t = O.fisher_pair(np.ascontiguousarray(G1.T), np.ascontiguousarray(G2.T), ROWS, COLS, n_seg, seg_len, 3.0)
    np.testing.assert_allclose(f_t, f, rtol=1e-14)


# ---------------------------------------------------------------------------
# Aligned selection (Definition 1)
# ---------------------------------------------------------------------------

def brute_force_topk(score, k):
    """rank(j) = #{i : s_i > s_j or (s_i == s_j and i < j)}; keep rank < k."""
    n = len(score)
    keep = []
    for j in range(n):
        rank = sum(1 for i in range(n) if score[i] > score[j] or (score[i] == score[j] and i < j))
        if rank < k:
            keep.append(j)
    return keep


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_select_matches_brute_force_with_ties(dtype):
    r = rng(8)
    n_seg, seg_len = 5, 17
    # few distinct values -> many exact ties
    s = r.integers(0, 4, size=n_seg * seg_len).astype(dtype) / 4
    k = [1, 17, 8, 9, 3]
    kept = O.select_topk(s, n_seg, seg_len, k)
    exp = []
    for i in range(n_seg):
        exp += [i * seg_len + j for j in brute_force_topk(s[i * seg_len:(i + 1) * seg_len], k[i])]
    assert kept.tolist() == exp


def test_select_all_equal_keeps_lowest_indices_and_counts():
    s = np.full(3 * 10, 0.25)
    kept = O.select_topk(s, 3, 10, [4, 10, 1])
    assert kept.tolist() == [0, 1, 2, 3] + list(range(10, 20)) + [20]


def test_select_keeps_exactly_k_ascending_inside_segment():
    r = rng(9)
    n_seg, seg_len = 16, 64
    s = r.random(n_seg * seg_len)
    k = r.integers(1, seg_len + 1, size=n_seg)
    kept = O.select_topk(s, n_seg, seg_len, k)
    off = 0
    for i in range(n_seg):
        part = kept[off:off + k[i]]
        assert np.all(np.diff(part) > 0)
        assert part.min() >= i * seg_len and part.max() < (i + 1) * seg_len
        # everything kept scores at least as high as everything dropped
        dropped = np.setdiff1d(np.arange(i * seg_len, (i + 1) * seg_len), part)
        if len(dropped):
            assert s[part].min() >= s[dropped].max()
        off += k[i]
    assert off == kept.size


def test_single_removal_is_frobenius_optimal_by_brute_force():
    # Proposition 1: removing argmin_j ||a_j|| ||b_j|| gives error exactly min_j ||a_j|| ||b_j||,
    # and no other single aligned removal does better.
    r = rng(10)
    for trial in range(5):
        m, n, p = 6, 9, 5
        A = r.standard_normal((m, n)); B = r.standard_normal((n, p))
        raw, ups = O.score_pair(A, B, COLS, ROWS, 1, n)
        errs = []
        for j in range(n):
            kept = [i for i in range(n) if i != j]
            e = O.frob_removed(A, B, kept, kept)
            errs.append(e)
            # ||a b^T||_F = ||a|| ||b||, and the oracle's error agrees with a library product
            assert abs(e - np.linalg.norm(A[:, j]) * np.linalg.norm(B[j, :])) < 1e-12
            assert abs(e - np.linalg.norm(A @ B - A[:, kept] @ B[kept, :])) < 1e-12
        jstar = int(np.argmin(errs))
        assert O.coupled_single(A, B) == jstar
        kept = O.select_topk(ups, 1, n, [n - 1]).tolist()
        assert kept == [i for i in range(n) if i != jstar]
        np.testing.assert_allclose(raw, errs, rtol=1e-12)


def test_exhaustive_subsets_tiny_pairs():
    r = rng(11)
    m, d, p = 12, 9, 4
    for k in (3, 5, 8):
        # general matrices: the kept set minimises the sum of removed raw scores (the bound the method ranks by)
        A = r.standard_normal((m, d)); B = r.standard_normal((d, p))
        raw, ups = O.score_pair(A, B, COLS, ROWS, 1, d)
        kept = tuple(O.select_topk(ups, 1, d, [k]).tolist())
        best = min(itertools.combinations(range(d), k), key=lambda S: sum(raw[j] for j in range(d) if j not in S))
        assert kept == best
        # orthogonal columns in A: cross terms vanish and the same set minimises the true Frobenius error
        Q, _ = np.linalg.qr(r.standard_normal((m, d)))
        Ao = Q * r.uniform(0.5, 2.0, size=d)[None, :]
        raw_o, ups_o = O.score_pair(Ao, B, COLS, ROWS, 1, d)
        kept_o = tuple(O.select_topk(ups_o, 1, d, [k]).tolist())
        best_o = min(itertools.combinations(range(d), k),
                     key=lambda S: np.linalg.norm(Ao @ B - Ao[:, list(S)] @ B[list(S), :]))
        assert kept_o == best_o


def test_multi_removal_error_closed_form():
    # ||A B - A_c B_c||_F^2 = sum_{i,j in R} (a_i . a_j)(b_i . b_j), R the removed set
    r = rng(12)
    A = r.standard_normal((7, 10)); B = r.standard_normal((10, 6))
    kept = [0, 2, 3, 7, 9]
    R = [j for j in range(10) if j not in kept]
    e = O.frob_removed(A, B, kept, kept)
    GA = A[:, R].T @ A[:, R]; GB = B[R, :] @ B[R, :].T
    assert abs(e ** 2 - (GA * GB).sum()) < 1e-10


def test_mismatch_worked_example_from_paper():
    line = [l for l in open(os.path.join(GOLDEN, "mismatch_example.txt")) if not l.startswith("#")][0]
    head, keepA, keepB, terms = [f.strip() for f in line.split("|")]
    n, kstar, lstar = map(int, head.split())
    keepA = [int(x) - 1 for x in keepA.split()]
    keepB = [int(x) - 1 for x in keepB.split()]
    r = rng(13)
    A = r.standard_normal((4, n)); B = r.standard_normal((n, 5))
    A[:, kstar - 1] *= 0.01                # a_1 is the smallest column
    B[lstar - 1, :] *= 0.01                # b_2 is the smallest row
    ks, ls = O.individual_single(A, B)
    assert (ks + 1, ls + 1) == (kstar, lstar)
    assert [i for i in range(n) if i != ks] == keepA and [i for i in range(n) if i != ls] == keepB
    delta = np.zeros((4, 5))
    for t in terms.split():
        sign, ia, ib = t.split(":")
        delta += (1.0 if sign == "+" else -1.0) * np.outer(A[:, int(ia) - 1], B[int(ib) - 1, :])
    assert abs(O.frob_removed(A, B, keepA, keepB) - np.linalg.norm(delta)) < 1e-12


def _a4_rows():
    rows = {}
    for l in open(os.path.join(GOLDEN, "appendix_a4_frobenius_table.txt")):
        if l.startswith("#") or not l.strip():
            continue
        n, d1, d2, p = l.split()
        rows[int(n)] = (float(d1), float(d2), float(p))
    return rows


@pytest.mark.parametrize("n,trials", [(100, 1000), (500, 300), (1000, 24)])
def test_appendix_a4_table_statistics(n, trials):
    """i.i.d. N(0,1) entries reproduce the printed means (the paper does not state the distribution)."""
    d1_ref, d2_ref, p_ref = _a4_rows()[n]
    r = rng(1000 + n)
    d1s, d2s = [], []
    for t in range(trials):
        A = r.standard_normal((n, n)); B = r.standard_normal((n, n))
        j = O.coupled_single(A, B)
        ks, ls = O.individual_single(A, B)
        raw, _ = O.score_pair(A, B, COLS, ROWS, 1, n)
        d1 = raw[j]
        keepA = np.delete(np.arange(n), ks); keepB = np.delete(np.arange(n), ls)
        if n == 100 and t < 10:
            # the oracle's own error routine, checked against the library product
            kept = np.delete(np.arange(n), j)
            assert abs(O.frob_removed(A, B, kept, kept) - d1) < 1e-9
            d2 = O.frob_removed(A, B, keepA, keepB)
            assert abs(d2 - np.linalg.norm(A @ B - A[:, keepA] @ B[keepB, :])) < 1e-8
        else:
            d2 = np.linalg.norm(A @ B - A[:, keepA] @ B[keepB, :])
        d1s.append(d1); d2s.append(d2)
    d1s, d2s = np.array(d1s), np.array(d2s)
    assert abs(d1s.mean() / d1_ref - 1.0) < 0.03
    assert abs(d2s.mean() / d2_ref - 1.0) < (0.05 if trials >= 300 else 0.25)
    p = 100.0 * np.mean(d1s < d2s)
    assert p >= p_ref - 1.5


# ---------------------------------------------------------------------------
# Compaction
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_compact_matches_index_select_and_zero_pads(dtype):
    g = torch.Generator().manual_seed(14)
    W1 = torch.randn(10, 24, generator=g).to(dtype); W2 = torch.randn(24, 7, generator=g).to(dtype)
    kept = [0, 3, 4, 11, 17, 23, 20][:6]
    kept = sorted(kept)
    idx = torch.tensor(kept)
    c1 = O.compact(W1, COLS, kept, ld_out=8)
    assert c1.shape == (10, 8)
    assert torch.equal(c1[:, :6], W1.index_select(1, idx)) and torch.all(c1[:, 6:] == 0)
    c2 = O.compact(W2, ROWS, kept, ld_out=8)
    assert c2.shape == (6, 8)
    assert torch.equal(c2[:, :7], W2.index_select(0, idx)) and torch.all(c2[:, 7:] == 0)
    b = torch.randn(24, generator=g).to(dtype)
    assert torch.equal(O.compact(b, COLS, kept), b[idx])


def test_restricted_product_invariant():
    # compacted W_1^c W_2^c equals the full product restricted to the kept index set, per head for QK
    r = rng(15)
    h, dh, dm = 3, 8, 24
    D = h * dh
    WQ = torch.from_numpy(r.standard_normal((dm, D))); WK = torch.from_numpy(r.standard_normal((dm, D)))
    _, ups = O.score_pair(WQ, WK, COLS, COLS, h, dh)
    k = [3, 8, 5]
    kept = O.select_topk(ups, h, dh, k)
    WQc = O.compact(WQ, COLS, kept).numpy(); WKc = O.compact(WK, COLS, kept).numpy()
    off = 0
    for i in range(h):
        ki = kept[off:off + k[i]]
        full = sum(np.outer(WQ[:, j].numpy(), WK[:, j].numpy()) for j in ki)
        np.testing.assert_allclose(WQc[:, off:off + k[i]] @ WKc[:, off:off + k[i]].T, full, rtol=1e-12, atol=1e-12)
        mask = np.zeros(D); mask[ki] = 1.0
        np.testing.assert_allclose(full, (WQ.numpy() * mask) @ WK.numpy().T, rtol=1e-12, atol=1e-12)
        off += k[i]
