"""Pins of the oracle's rotation-pair (rotary position embedding) score and removal.

With RoPE the coupled matrix is W_Q P_t P_s^T W_K^T (Eq. "self-attention-rope"): P rotates the shared index in
2 x 2 blocks.  The pins: the pair score does not depend on the rotations (so "incorporating the position
matrices" gives one score for all positions), the per-index score does; a pair whose second member is zero
scores like its first member alone; removal keeps whole pairs and the compacted matrices still carry the
storage convention of the pairs, shown by the attention logits of random positions.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O


@pytest.fixture(scope="module", autouse=True)
def _build():
    O.build()


def members(u, d_h, mode):
    return (2 * u, 2 * u + 1) if mode == 1 else (u, u + d_h // 2)


def rotate_pairs(W, angles, d_h, mode):
    """W (d_m x h*d_h) with every rotation pair of every head rotated by its own angle (columns mixed in pairs)."""
    W = W.clone()
    h = W.shape[1] // d_h
    for i in range(h):
        for u in range(d_h // 2):
            a, b = members(u, d_h, mode)
            a += i * d_h; b += i * d_h
            c, s = np.cos(angles[i, u]), np.sin(angles[i, u])
            wa, wb = W[:, a].clone(), W[:, b].clone()
            W[:, a] = c * wa - s * wb
            W[:, b] = s * wa + c * wb
    return W


@pytest.mark.parametrize("mode", [1, 2])
def test_pair_score_is_the_same_at_every_position(mode):
    g = torch.Generator().manual_seed(1)
    d_m, h, d_h = 24, 3, 8
    WQ = torch.randn(d_m, h * d_h, generator=g, dtype=torch.float64)
    WK = torch.randn(d_m, h * d_h, generator=g, dtype=torch.float64)
    raw0, ups0 = O.score_pair(WQ, WK, O.SHARED_COLS, O.SHARED_COLS, h, d_h, rope=mode)
    r = np.random.default_rng(2)
    for _ in range(3):
        WQr = rotate_pairs(WQ, r.uniform(0, 6.28, size=(h, d_h // 2)), d_h, mode)
        WKr = rotate_pairs(WK, r.uniform(0, 6.28, size=(h, d_h // 2)), d_h, mode)
        raw1, ups1 = O.score_pair(WQr, WKr, O.SHARED_COLS, O.SHARED_COLS, h, d_h, rope=mode)
        assert np.allclose(raw1, raw0, rtol=1e-12, atol=0) and np.allclose(ups1, ups0, rtol=1e-12, atol=0)
        # the per-index score of Eq. "l2norm" is not: it would depend on the position
        _, plain0 = O.score_pair(WQ, WK, O.SHARED_COLS, O.SHARED_COLS, h, d_h)
        _, plain1 = O.score_pair(WQr, WKr, O.SHARED_COLS, O.SHARED_COLS, h, d_h)
        assert not np.allclose(plain1, plain0, rtol=1e-3)
    # both members carry the pair's value and the units of a head have unit l2 norm
    for i in range(h):
        seg = ups0[i * d_h:(i + 1) * d_h]
        for u in range(d_h // 2):
            a, b = members(u, d_h, mode)
            assert seg[a] == seg[b]
        firsts = np.array([seg[members(u, d_h, mode)[0]] for u in range(d_h // 2)])
        assert abs((firsts ** 2).sum() - 1.0) < 1e-12


@pytest.mark.parametrize("mode", [1, 2])
def test_reduces_to_the_plain_score_when_second_members_are_zero(mode):
    g = torch.Generator().manual_seed(3)
    d_m, d_h = 16, 12
    WQ = torch.randn(d_m, d_h, generator=g, dtype=torch.float64)
    WK = torch.randn(d_m, d_h, generator=g, dtype=torch.float64)
    seconds = [members(u, d_h, mode)[1] for u in range(d_h // 2)]
    firsts = [members(u, d_h, mode)[0] for u in range(d_h // 2)]
    WQ[:, seconds] = 0; WK[:, seconds] = 0
    raw_r, ups_r = O.score_pair(WQ, WK, O.SHARED_COLS, O.SHARED_COLS, 1, d_h, rope=mode)
    raw_p, _ = O.score_pair(WQ[:, firsts].contiguous(), WK[:, firsts].contiguous(), O.SHARED_COLS, O.SHARED_COLS, 1, d_h // 2)
    assert np.allclose(raw_r[firsts], raw_p, rtol=1e-13) and np.allclose(raw_r[seconds], raw_p, rtol=1e-13)


def rope_matrix(pos, thetas, mode):
    """P_pos for len(thetas) rotation pairs stored in the convention of `mode` (blocks as the paper prints them)."""
    n = 2 * len(thetas)
    P = np.zeros((n, n))
    for u, th in enumerate(thetas):
        a, b = members(u, n, mode)
        c, s = np.cos(pos * th), np.sin(pos * th)
        P[a, a] = c; P[a, b] = s; P[b, a] = -s; P[b, b] = c
    return P


@pytest.mark.parametrize("mode", [1, 2])
def test_kept_pairs_keep_the_rope_structure(mode):
    """Logits x_q W_Q P_t P_s^T W_K^T x_k restricted to the kept pairs == the same expression on the compacted
    matrices with position matrices built from the kept pairs' frequencies, in the same storage convention."""
    r = np.random.default_rng(5)
    d_m, d_h, k = 20, 16, 10
    WQ = r.standard_normal((d_m, d_h)); WK = r.standard_normal((d_m, d_h))
    _, ups = O.score_pair(torch.from_numpy(WQ), torch.from_numpy(WK), O.SHARED_COLS, O.SHARED_COLS, 1, d_h, rope=mode)
    kept = O.select_rotation_pairs(ups.astype(np.float32), 1, d_h, [k], mode)
    assert kept.size == k and (np.diff(kept) > 0).all()
    theta = 10000.0 ** (-2.0 * np.arange(d_h // 2) / d_h)
    units = sorted({(j // 2) if mode == 1 else (j % (d_h // 2)) for j in kept})
    assert len(units) == k // 2                                             # whole pairs
    for u in units:
        a, b = members(u, d_h, mode)
        assert a in kept and b in kept
    # the kept units are the k/2 best ones
    unit_score = np.array([ups[members(u, d_h, mode)[0]] for u in range(d_h // 2)])
    assert set(units) == set(np.argsort(-unit_score, kind="stable")[:k // 2].tolist())
    xq, xk = r.standard_normal(d_m), r.standard_normal(d_m)
    WQc, WKc = WQ[:, kept], WK[:, kept]
    for t, s_ in ((3, 7), (100, 1)):
        q = xq @ WQ @ rope_matrix(t, theta, mode)
        kk = xk @ WK @ rope_matrix(s_, theta, mode)
        want = float(q[kept] @ kk[kept])
        Pt, Ps = rope_matrix(t, theta[units], mode), rope_matrix(s_, theta[units], mode)
        got = float((xq @ WQc @ Pt) @ (xk @ WKc @ Ps))
        assert abs(got - want) <= 1e-10 * max(1.0, abs(want))


def test_select_rotation_pairs_ties_and_counts():
    u = np.array([5, 5, 1, 1, 5, 5, 3, 3], dtype=np.float32)               # interleaved: units 0, 2 tie
    assert O.select_rotation_pairs(u, 1, 8, [2], 1).tolist() == [0, 1]
    assert O.select_rotation_pairs(u, 1, 8, [4], 1).tolist() == [0, 1, 4, 5]
    assert O.select_rotation_pairs(u, 1, 8, [6], 1).tolist() == [0, 1, 4, 5, 6, 7]
    v = np.array([5, 1, 5, 3, 5, 1, 5, 3], dtype=np.float32)               # halves: unit u = (u, u + 4)
    assert O.select_rotation_pairs(v, 1, 8, [2], 2).tolist() == [0, 4]
    assert O.select_rotation_pairs(v, 1, 8, [4], 2).tolist() == [0, 2, 4, 6]
    assert O.select_rotation_pairs(v, 1, 8, [0], 2).size == 0
