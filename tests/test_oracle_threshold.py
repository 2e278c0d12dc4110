"""Pins of the oracle's Algorithm 1 steps: the cumulative-threshold loop and the top-K pair choice.

The loop is pinned by exactly representable closed forms, by an independent characterisation evaluated with
exact summation (math.fsum) on random inputs, and by the invariances the rule must have.
"""
import math

import numpy as np
import pytest

from oracle import oracle as O


@pytest.fixture(scope="module", autouse=True)
def _build():
    O.build()


def test_uniform_scores_exact():
    # eight scores of 1/8, theta = 3/4 of the mass: 1 > .75, .875 > .75, .75 is not > .75 -> six stay
    u = np.full(8, 0.125, dtype=np.float32)
    assert O.threshold_counts(u, 1, 8, 0.75, l1=True)[0] == 6
    # compared as stored (total = 1): same numbers, same answer
    assert O.threshold_counts(u, 1, 8, 0.75, l1=False)[0] == 6


def test_geometric_scores_closed_form():
    # scores 2^-1 .. 2^-20: the k largest sum to 1 - 2^-k exactly; 1 - 2^-3 <= 0.9 < 1 - 2^-4
    u = np.array([2.0 ** -(i + 1) for i in range(20)], dtype=np.float32)
    assert O.threshold_counts(u, 1, 20, 0.9, l1=False)[0] == 3
    assert O.threshold_counts(u[::-1].copy(), 1, 20, 0.9, l1=False)[0] == 3      # order of storage does not matter
    # as a share of the mass (total = 1 - 2^-20): 0.9 * total is still between the same two prefix sums
    assert O.threshold_counts(u, 1, 20, 0.9, l1=True)[0] == 3
    # 1 - 2^-k <= 0.5 only for k = 1
    assert O.threshold_counts(u, 1, 20, 0.5, l1=False)[0] == 1


def test_matches_prefix_characterisation_with_exact_sums():
    # the loop stops at the largest k whose k largest scores sum to at most theta * total
    r = np.random.default_rng(3)
    for trial in range(40):
        d = int(r.integers(2, 200))
        u = r.random(d).astype(np.float32) ** 3
        theta = float(r.uniform(0.05, 0.999))
        s = sorted((float(x) for x in u), reverse=True)
        total = math.fsum(s)
        budget = theta * total
        prefix = [math.fsum(s[:k]) for k in range(d + 1)]
        if min(abs(p - budget) for p in prefix) < 1e-9 * total:
            continue                                   # decision too close to call between summation orders
        want = max(k for k in range(d + 1) if prefix[k] <= budget)
        want = max(want, 1)
        assert O.threshold_counts(u, 1, d, theta, l1=True, k_min=1)[0] == want


def test_limits_and_monotonicity():
    r = np.random.default_rng(5)
    u = r.random(3 * 64).astype(np.float32)
    assert (O.threshold_counts(u, 3, 64, 1.0, l1=True) == 64).all()          # the whole mass may stay
    assert (O.threshold_counts(u, 3, 64, 1e-9, l1=True, k_min=4) == 4).all()  # never below k_min
    prev = np.zeros(3, dtype=np.int32)
    for theta in np.linspace(0.05, 1.0, 20):
        k = O.threshold_counts(u, 3, 64, float(theta), l1=True)
        assert (k >= prev).all()
        prev = k
    z = np.zeros(16, dtype=np.float32)
    assert O.threshold_counts(z, 1, 16, 0.9, l1=True)[0] == 16              # nothing exceeds a zero budget


def test_invariances():
    r = np.random.default_rng(9)
    u = (r.random(2 * 96).astype(np.float32) + 0.01)
    k = O.threshold_counts(u, 2, 96, 0.8, l1=True)
    # a share of the mass does not change when every score is doubled (exact in fp32)
    assert (O.threshold_counts(2 * u, 2, 96, 0.8, l1=True) == k).all()
    # nor when the indices of a segment are permuted
    v = u.copy().reshape(2, 96)
    v[0] = v[0][r.permutation(96)]
    v[1] = v[1][r.permutation(96)]
    assert (O.threshold_counts(v.reshape(-1), 2, 96, 0.8, l1=True) == k).all()
    # segments that were not chosen keep everything
    assert (O.threshold_counts(u, 2, 96, 0.8, l1=True, chosen=[0, 1]) == np.array([96, k[1]])).all()


def test_removed_indices_are_the_smallest():
    r = np.random.default_rng(11)
    u = r.random(128).astype(np.float32)
    k = int(O.threshold_counts(u, 1, 128, 0.7, l1=True)[0])
    kept = O.select_topk(u, 1, 128, [k])
    removed = np.setdiff1d(np.arange(128), kept)
    assert u[removed].max() <= u[kept].min()
    assert float(u[kept].astype(np.float64).sum()) <= 0.7 * float(u.astype(np.float64).sum()) * (1 + 1e-12)
    # one more index would exceed the budget
    if k < 128:
        nxt = np.sort(u)[::-1][:k + 1].astype(np.float64).sum()
        assert nxt > 0.7 * float(u.astype(np.float64).sum()) * (1 - 1e-12)


def test_choose_pairs_against_a_stable_library_sort():
    r = np.random.default_rng(13)
    f = r.random(50).astype(np.float32)
    f[7] = f[3]; f[20] = f[3]                                    # ties: lower index first
    for m in (0, 1, 15, 50):
        want = np.zeros(50, dtype=np.int32)
        want[np.argsort(f, kind="stable")[:m]] = 1
        assert (O.choose_pairs(f, m) == want).all()
    g = np.array([3, 1, 1, 2], dtype=np.float32)
    assert O.choose_pairs(g, 1).tolist() == [0, 1, 0, 0]
    assert O.choose_pairs(g, 2).tolist() == [0, 1, 1, 0]


def test_rotation_pairs_are_thresholded_as_units():
    r = np.random.default_rng(17)
    half = 24
    unit = r.random(half).astype(np.float32)
    inter = np.repeat(unit, 2)                       # members (2u, 2u+1) carry the pair's score
    halves = np.concatenate([unit, unit])            # members (u, u + half)
    for theta in (0.3, 0.8, 0.95):
        k_units = int(O.threshold_counts(unit, 1, half, theta, l1=True, k_min=1)[0])
        assert O.threshold_counts(inter, 1, 2 * half, theta, l1=True, k_min=1, rope=1)[0] == 2 * k_units
        assert O.threshold_counts(halves, 1, 2 * half, theta, l1=True, k_min=2, rope=2)[0] == 2 * k_units
    assert O.threshold_counts(inter, 1, 2 * half, 1e-9, l1=True, k_min=3, rope=1)[0] == 4      # k_min in whole pairs
