"""Pins for the fixed-budget selector (Section 4.1) and the forced-position variant of the oracle."""
import numpy as np
import pytest

from oracle import rtp_oracle as orc


@pytest.mark.parametrize("n,k", [(1, 1), (7, 3), (64, 64), (200, 17), (1000, 4096), (5000, 4096)])
def test_topk_is_the_k_largest_on_distinct_scores(n, k):
    rng = np.random.default_rng(100 + n + k)
    s = rng.permutation(n).astype(np.float32) * 0.37 - 11.0   # all different
    ids, c, thr, tie_last = orc.topk_select(s, k)
    assert c == min(k, n) == ids.size
    if c < n:
        want = np.sort(np.argpartition(-s, c - 1)[:c])   # a library routine that does not sort the row
        assert np.array_equal(ids, want)
        rest = np.setdiff1d(np.arange(n), ids)
        assert s[ids].min() > s[rest].max()
    else:
        assert np.array_equal(ids, np.arange(n))
    assert thr == s[ids].min()
    assert s[tie_last] == thr and tie_last in set(ids.tolist())


def test_topk_equal_scores_go_to_the_smaller_positions():
    s = np.zeros(50, dtype=np.float32)
    ids, c, thr, tie_last = orc.topk_select(s, 20)
    assert np.array_equal(ids, np.arange(20)) and c == 20 and thr == 0.0 and tie_last == 19
    # two values: every key of the larger value, then the first ones of the smaller
    s = np.where(np.arange(50) % 5 == 0, 1.0, 0.0).astype(np.float32)   # ten ones
    ids, c, thr, tie_last = orc.topk_select(s, 14)
    ones = np.arange(0, 50, 5)
    zeros_first = np.setdiff1d(np.arange(50), ones)[:4]
    assert np.array_equal(ids, np.sort(np.concatenate([ones, zeros_first])))
    assert thr == 0.0 and tie_last == int(zeros_first.max())
    # the cut falls inside the larger value
    ids, c, thr, tie_last = orc.topk_select(s, 3)
    assert np.array_equal(ids, ones[:3]) and thr == 1.0 and tie_last == 10


def test_topk_brute_force_tiny():
    # among all subsets of size k, the one taken has the largest score sum and, among those, the smallest positions
    from itertools import combinations
    rng = np.random.default_rng(5)
    for _ in range(30):
        n = int(rng.integers(2, 9))
        k = int(rng.integers(1, n + 1))
        s = rng.integers(0, 3, size=n).astype(np.float32)   # many ties
        ids, c, _, _ = orc.topk_select(s, k)
        best = max(combinations(range(n), k), key=lambda t: (float(s[list(t)].sum()), [-i for i in t]))
        assert tuple(ids.tolist()) == best


def test_topk_agrees_with_topp_at_its_own_mass():
    # Top-P with p = the mass of the k largest keys takes exactly those keys (distinct scores).
    rng = np.random.default_rng(9)
    s = (rng.standard_normal(300) * 2.0).astype(np.float32)
    for k in (1, 5, 60, 299):
        ids, c, _, _ = orc.topk_select(s, k)
        mass = orc.set_mass(s, ids)
        got = orc.topp_select(s, mass * (1 - 1e-12))[0]
        assert np.array_equal(got, ids)


def test_topk_rejects_bad_arguments():
    with pytest.raises(ValueError):
        orc.topk_select(np.zeros(4, dtype=np.float32), 0)
    with pytest.raises(ValueError):
        orc.topk_select(np.zeros(0, dtype=np.float32), 3)


@pytest.mark.parametrize("m,ns,nr", [(0, 4, 16), (3, 4, 16), (19, 4, 16), (20, 4, 16), (1000, 4, 16), (1000, 0, 0),
                                      (1000, 0, 7), (1000, 5, 0), (10, 8, 8)])
def test_forced_positions_closed_form(m, ns, nr):
    f = orc.forced_tokens(m, ns, nr)
    n = m + 1
    assert f.size == min(n, ns + nr)             # the two ranges overlap exactly when the row is shorter than both
    assert np.all((f >= 0) & (f <= m))
    assert np.all(np.diff(f) > 0)
    assert set(range(min(ns, n))) <= set(f.tolist())
    assert set(range(max(0, n - nr), n)) <= set(f.tolist())
    for j in f.tolist():
        assert j < ns or j > m - nr


def test_with_forced_is_a_union():
    rng = np.random.default_rng(3)
    s = rng.standard_normal(500).astype(np.float32)
    ids = orc.topp_select(s, 0.5)[0]
    u = orc.with_forced(ids, 499, 4, 32)
    assert set(ids.tolist()) <= set(u.tolist())
    assert set(u.tolist()) - set(ids.tolist()) <= set(orc.forced_tokens(499, 4, 32).tolist())
    assert np.array_equal(orc.with_forced(ids, 499, 0, 0), ids)
    assert np.array_equal(orc.with_forced(u, 499, 4, 32), u)              # idempotent
    assert np.array_equal(orc.with_forced(np.arange(500), 499, 4, 32), np.arange(500))
