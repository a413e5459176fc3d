"""Pins of the block-wise top-p selection (Section 3.4) against what the mathematics fixes."""
import itertools

import numpy as np
import pytest

from oracle import rtp_oracle as orc


def test_equal_blocks_take_ceil_p_times_n():
    # every block carries the same pair (m_b, l_b): mass 1/N_b each, taken in index order
    rng = np.random.default_rng(0)
    blk = rng.standard_normal(64).astype(np.float32)
    for n_b, p in [(10, 0.85), (7, 0.5), (16, 0.99), (3, 0.4)]:        # (p never a multiple of 1 / N_b)
        s = np.tile(blk, n_b)
        ids, k, mass, thr, _, _ = orc.topp_select_blocks(s, p)
        want = int(np.ceil(p * n_b))
        assert k == want and list(ids) == list(range(want))
        assert abs(mass - want / n_b) < 1e-12 and thr == blk.max()


def test_one_dominant_block():
    rng = np.random.default_rng(1)
    s = rng.standard_normal(64 * 9).astype(np.float32)
    s[64 * 5 + 17] = 30.0
    ids, k, mass, thr, _, _ = orc.topp_select_blocks(s, 0.9)
    assert list(ids) == [5] and k == 1 and mass > 0.999 and thr == np.float32(30.0)


def test_block_of_one_is_the_token_rule():
    rng = np.random.default_rng(2)
    for trial in range(20):
        s = (2.0 * rng.standard_normal(200)).astype(np.float32)
        p = float(rng.uniform(0.05, 0.99))
        a = orc.topp_select(s, p)
        b = orc.topp_select_blocks(s, p, block=1)
        assert list(a[0]) == list(b[0]) and a[1] == b[1] and abs(a[2] - b[2]) < 1e-12 and a[3] == b[3]


def test_block_pairs_are_the_log_sum_exp_of_the_block():
    rng = np.random.default_rng(3)
    s = (3.0 * rng.standard_normal(64 * 4 + 11)).astype(np.float32)      # ragged last block
    m, l = orc.block_lse(s)
    assert m.shape == (5,)
    for b in range(5):
        blk = s[64 * b: 64 * (b + 1)].astype(np.float64)
        assert m[b] == blk.max()
        assert abs(np.log(l[b]) + float(m[b]) - np.log(np.sum(np.exp(blk)))) < 1e-12
    # block masses add up to the row's softmax: mass of a block = sum of its tokens' probabilities
    _, _, P = orc.softmax_mass(s)
    w = l * np.exp(m.astype(np.float64) - float(m.max()))
    for b in range(5):
        assert abs(w[b] / w.sum() - P[64 * b: 64 * (b + 1)].sum()) < 1e-12


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_prefix_in_max_order(seed):
    # among all prefixes of the (m_b descending) order the selection is the shortest one reaching p,
    # and no shorter set of blocks that respects the order exists: checked by enumeration
    rng = np.random.default_rng(10 + seed)
    n_b, blk = 6, 4
    s = (1.5 * rng.standard_normal(n_b * blk)).astype(np.float32)
    p = float(rng.uniform(0.3, 0.95))
    ids, k, mass, thr, order, cum = orc.topp_select_blocks(s, p, block=blk)
    _, _, P = orc.softmax_mass(s)
    bm = np.array([P[blk * b: blk * (b + 1)].sum() for b in range(n_b)])
    mx = np.array([s[blk * b: blk * (b + 1)].max() for b in range(n_b)])
    best = None
    for r in range(1, n_b + 1):
        for sub in itertools.combinations(range(n_b), r):
            rest = [b for b in range(n_b) if b not in sub]
            closed = all(mx[a] > mx[b] or (mx[a] == mx[b] and a < b) for a in sub for b in rest)   # a prefix of the order
            if closed and bm[list(sub)].sum() >= p:
                best = sub
                break
        if best:
            break
    assert best is not None and sorted(best) == list(ids) and len(best) == k
    assert abs(bm[list(best)].sum() - mass) < 1e-12


def test_p_one_keeps_every_block_and_band_classification():
    rng = np.random.default_rng(5)
    s = rng.standard_normal(64 * 6 + 3).astype(np.float32)
    ids, k, mass, _, _, _ = orc.topp_select_blocks(s, 1.0)
    assert k == 7 and abs(mass - 1.0) < 1e-12
    mand, forb = orc.classify_blocks_against_band(s, 0.8)
    sel = set(orc.topp_select_blocks(s, 0.8)[0].tolist())
    assert mand <= sel and not (forb & sel)
    toks = orc.block_token_set(sorted(sel), 64 * 6 + 2)
    assert set((toks // 64).tolist()) == sel and toks.max() <= 64 * 6 + 2
