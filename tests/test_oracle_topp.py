"""Pins for the oracle's top-p selection (Eq. 5): brute force, closed forms, invariants."""
import itertools
import math
import os
from statistics import NormalDist

import numpy as np
import pytest

from oracle import rtp_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


@pytest.mark.parametrize("seed", range(12))
def test_bruteforce_all_subsets(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 13))
    s = (rng.standard_normal(L) * rng.uniform(0.2, 4.0)).astype(np.float32)
    p = float(rng.uniform(0.05, 0.999))
    ids, k_star, mass, thr, order, cum = orc.topp_select(s, p)
    e = np.exp(s.astype(np.float64) - s.astype(np.float64).max())
    P = e / e.sum()
    # smallest subset of ANY kind whose mass reaches p
    best = None
    for k in range(1, L + 1):
        top = max(sum(P[list(c)]) for c in itertools.combinations(range(L), k))
        if top >= p:
            best = (k, top)
            break
    assert best is not None and best[0] == k_star
    assert mass == pytest.approx(best[1], rel=1e-12)          # and it is the heaviest such subset
    assert mass >= p
    if k_star > 1:
        assert cum[k_star - 2] < p                              # one token fewer is not enough
    assert len(ids) == k_star and np.all(np.diff(ids) > 0)
    assert thr == s[ids].min()


def test_equal_scores_take_lowest_indices():
    for L, p in [(100, 0.9), (7, 0.5), (64, 0.95), (1, 0.9), (10, 0.1)]:
        s = np.full(L, 3.25, np.float32)
        ids, k_star, mass, thr, _, _ = orc.topp_select(s, p)
        # k/L >= p; guard the product against 1-ulp noise
        want = min(L, max(1, math.ceil(p * L - 1e-9)))
        assert k_star == want
        assert ids.tolist() == list(range(want))


def test_geometric_scores_golden():
    n = 40
    s = (-np.arange(n) * math.log(2.0)).astype(np.float32)
    for p, k in _rows(os.path.join(GOLDEN, "geometric_prefix_mass.txt")):
        ids, k_star, mass, thr, _, _ = orc.topp_select(s, float(p) - 1e-9)
        assert k_star == int(k)
        assert ids.tolist() == list(range(int(k)))
        assert mass == pytest.approx(1 - 2.0 ** (-int(k)), rel=1e-6)


def test_one_dominant_score():
    rng = np.random.default_rng(3)
    s = rng.standard_normal(5000).astype(np.float32)
    s[1234] = 45.0
    ids, k_star, mass, thr, _, _ = orc.topp_select(s, 0.9)
    assert k_star == 1 and ids.tolist() == [1234] and thr == np.float32(45.0)


def test_two_tokens_holding_most_mass():
    # a concentrated row: two keys far above the rest are enough for p = 0.9
    s = np.zeros(35000, np.float32)
    s[17] = 14.0
    s[30000] = 14.2
    ids, k_star, mass, _, _, _ = orc.topp_select(s, 0.9)
    assert ids.tolist() == [17, 30000]
    hi = math.exp(float(np.float32(14.2)))
    z = math.exp(14.0) + hi + (35000 - 2)
    assert mass == pytest.approx((math.exp(14.0) + hi) / z, rel=1e-9)


@pytest.mark.parametrize("seed", range(5))
def test_invariants(seed):
    rng = np.random.default_rng(100 + seed)
    L = 777
    s = (rng.standard_normal(L) * 2.0).astype(np.float32)
    base = orc.topp_select(s, 0.9)[0]
    # adding a constant (exactly representable shift) changes nothing
    shifted = orc.topp_select((s.astype(np.float64) + 8.0), 0.9)[0]
    assert shifted.tolist() == base.tolist()
    # nested in p
    prev = set()
    for p in [0.1, 0.5, 0.8, 0.9, 0.99, 1.0]:
        cur = set(orc.topp_select(s, p)[0].tolist())
        assert prev <= cur
        prev = cur
    assert len(prev) == L                                    # p = 1 keeps everything
    # permuting the keys permutes the ids (scores distinct here)
    perm = rng.permutation(L)
    ids_p = orc.topp_select(s[perm], 0.9)[0]
    assert sorted(perm[ids_p].tolist()) == base.tolist()
    # never empty
    assert orc.topp_select(s, 1e-9)[1] == 1


def test_tie_break_prefers_smaller_index():
    s = np.array([1.0, 2.0, 2.0, 2.0, 0.0], np.float32)
    # masses: three equal heavy tokens; p small enough for one, two of them
    e = np.exp(s - 2.0)
    P = e / e.sum()
    ids1 = orc.topp_select(s, float(P[1]) * 0.99)[0]
    ids2 = orc.topp_select(s, float(P[1]) * 1.5)[0]
    assert ids1.tolist() == [1] and ids2.tolist() == [1, 2]


def test_gaussian_scores_selected_fraction():
    # iid N(0, sigma^2) scores: the mass profile is lognormal and the selected
    # fraction tends to 1 - Phi(sigma - Phi^-1(p)).
    nd = NormalDist()
    rng = np.random.default_rng(7)
    L = 1 << 18
    # (beyond sigma ~ 2.5 a finite sample's mass is dominated by a few extreme tokens and the
    # limit is approached too slowly to test)
    for sigma in (1.0, 1.5, 2.12):
        s = (rng.standard_normal(L) * sigma).astype(np.float32)
        k = orc.topp_select(s, 0.9)[1]
        want = 1.0 - nd.cdf(sigma - nd.inv_cdf(0.9))
        assert k / L == pytest.approx(want, rel=0.05)


def test_band_classification_consistent():
    rng = np.random.default_rng(11)
    s = (rng.standard_normal(4000) * 2.5).astype(np.float32)
    ids = set(orc.topp_select(s, 0.9)[0].tolist())
    mand, forb = orc.classify_against_band(s, 0.9)
    assert mand <= ids and not (forb & ids)
    assert orc.set_mass(s, ids) >= 0.9


def _geometric(n=60):
    # s_i = -i ln 2: softmax masses 2^-(i+1) / (1 - 2^-n); cumulative mass before token k is 1 - 2^-k
    return -np.arange(n, dtype=np.float64) * np.log(2.0)


def test_set_mass_closed_form_geometric():
    s = _geometric()
    for k in (1, 2, 4, 7, 20):
        assert orc.set_mass(s, range(k)) == pytest.approx(1.0 - 2.0 ** -k, abs=1e-12)
    # an arbitrary subset, given in any order and as any iterable
    assert orc.set_mass(s, [3, 1]) == pytest.approx(2.0 ** -2 + 2.0 ** -4, abs=1e-12)
    assert orc.set_mass(s, {0}) == pytest.approx(0.5, abs=1e-12)
    # normalised over the WHOLE row, whatever constant is added to the scores
    assert orc.set_mass(s + 37.5, range(4)) == pytest.approx(0.9375, abs=1e-12)
    assert orc.set_mass(s, range(len(s))) == pytest.approx(1.0, abs=1e-12)


def test_band_classification_closed_form_geometric():
    s = _geometric().astype(np.float32)
    n = len(s)
    # p = 0.9: cumulative mass before tokens 0..3 is 0, .5, .75, .875 (mandatory); before token 4 it is .9375
    mand, forb = orc.classify_against_band(s, 0.9)
    assert mand == {0, 1, 2, 3}
    assert forb == set(range(4, n))
    # the mass before token 4 is 0.9375: it is mandatory / optional / forbidden according to where p lies
    # relative to 0.9375 -+ 1e-4; token 3 (before: .875) and token 5 (before: .96875) never change class
    cases = [(+2e-4, "mandatory"), (+5e-5, "optional"), (-5e-5, "optional"), (-2e-4, "forbidden")]
    for delta, want in cases:
        mand, forb = orc.classify_against_band(s, 0.9375 + delta)
        got = "mandatory" if 4 in mand else "forbidden" if 4 in forb else "optional"
        assert got == want, (delta, got)
        assert {0, 1, 2, 3} <= mand and 5 in forb and 5 not in mand
        assert not (mand & forb)
    # the band argument is honoured: ten times wider makes token 4 optional in both outer cases,
    # a hundred times narrower leaves no optional token at +-5e-5
    for delta in (+2e-4, -2e-4):
        mand, forb = orc.classify_against_band(s, 0.9375 + delta, band=1e-3)
        assert 4 not in mand and 4 not in forb
    mand, forb = orc.classify_against_band(s, 0.9375 + 5e-5, band=1e-6)
    assert 4 in mand
    mand, forb = orc.classify_against_band(s, 0.9375 - 5e-5, band=1e-6)
    assert 4 in forb
    # every token is classified at most once and p = 1 makes every token mandatory
    mand, forb = orc.classify_against_band(s, 1.0)
    assert mand == set(range(n)) and forb == set()


def test_band_classification_uses_mass_before_inclusion():
    # two tokens of mass 0.6 / 0.4 (scores ln 0.6, ln 0.4): for p = 0.6 the first token alone reaches p; the
    # second has 0.6 before it, which is inside the band around p, so it may go either way; for p = 0.5 it is
    # forbidden, for p = 0.7 mandatory
    s = np.log(np.array([0.6, 0.4])).astype(np.float32)
    assert orc.classify_against_band(s, 0.6) == ({0}, set())
    assert orc.classify_against_band(s, 0.5) == ({0}, {1})
    assert orc.classify_against_band(s, 0.7) == ({0, 1}, set())


def test_rejects_bad_p():
    with pytest.raises(ValueError):
        orc.topp_select(np.zeros(4, np.float32), 0.0)
    with pytest.raises(ValueError):
        orc.topp_select(np.zeros(4, np.float32), float("nan"))
