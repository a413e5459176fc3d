"""GPU parity of the selectable variants of the decode selection, through the C ABI: the fixed-budget selector of
Section 4.1 (top-k) and forced sink / recent positions."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as gh
    return gh


def _run(wl, sel_stride=None, rows=None, attention=True, **variant):
    gh = _harness()
    dw = gh.DeviceWorkload(wl, sel_stride=sel_stride, **variant)
    dw.index_all_keys()
    qt = gh.check_queries(dw)
    sc = gh.check_scores(dw, qt, rows=rows)
    sel = dw.select()
    counts = gh.check_variant_selection(dw, sc, sel, rows=rows, **variant)
    if attention:
        out, lse = dw.sparse_decode()
        gh.check_sparse_attention(dw, sel, out, lse, rows=rows)
    assert dw.status_code() == rb.RTP_OK
    return dw, counts


def _ragged_config2():
    wl = synth.config_2(L=3000, batch=4, window=512)
    for b, cut in enumerate([0, 517, 1, 2049]):
        L = 3000 - cut
        wl.k[b], wl.v[b] = wl.k[b][:L], wl.v[b][:L]
        wl.seq_lens[b] = L
        wl.row_pos[b] = L - 1
    return wl


@pytest.mark.parametrize("k", [1, 7, 256, 2000])
def test_topk_ragged_batch(k):
    dw, counts = _run(_ragged_config2(), top_k=k)
    assert all(c == min(k, n) for c, _, n in counts)


def test_topk_not_smaller_than_the_row_takes_every_key():
    dw, counts = _run(_ragged_config2(), top_k=4096)
    assert all(c == n for c, _, n in counts)


@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 130, 1000])
def test_topk_ragged_lengths(L):
    _run(synth.config_1(L=L, n_needles=min(8, max(1, L // 4))), top_k=16)


def test_topk_cut_far_below_the_maximum():
    """Peaked scores (planted needles far above the bulk) and a budget that reaches deep into the bulk: the cut lies in
    the pooled last bin of the first histogram level."""
    wl = synth.config_1(L=4096, n_needles=8)
    wl.score_scale *= 4.0                                       # a colder temperature spreads the scores
    dw, counts = _run(wl, top_k=3000)
    sc = dw.scores()[0][0, 0, :4096]
    assert np.sort(sc)[-3000] < sc.max() - 32.0       # the input does what the test is about
    assert counts[0][0] == 3000


@pytest.mark.parametrize("L,k", [(100, 37), (4097, 1000), (9000, 4096), (9000, 8999)])
def test_topk_equal_scores_take_lowest_positions(L, k):
    gh = _harness()
    wl = synth.config_1(L=L)
    wl.k[0][:, 0, :] = wl.k[0][0, 0, :]                        # identical keys: every score ties
    dw = gh.DeviceWorkload(wl, top_k=k)
    dw.index_all_keys()
    sc = dw.scores()[0]
    assert np.all(sc[0, 0, :L] == sc[0, 0, 0])
    sel = dw.select()
    assert int(sel["cnt"][0, 0]) == k
    assert sorted(sel["idx"][0, 0, :k].cpu().numpy().tolist()) == list(range(k))
    assert int(sel["tie"][0, 0]) == k - 1
    gh.check_variant_selection(dw, sc, sel, top_k=k)


def test_topk_dense_cluster_of_near_equal_scores():
    wl = synth.config_1(L=20000, n_needles=4)
    K = wl.k[0]
    rng = np.random.default_rng(7)
    base = K[int(wl.notes["needles"][0]), 0].copy()
    for n in range(3000, 15000):
        k = base.copy()
        dims = rng.integers(0, 128, size=3)
        k[dims] ^= np.uint16(1)
        K[n, 0] = k
    _run(wl, sel_stride=20000, top_k=4096)
    _run(wl, sel_stride=20000, top_k=11000, attention=False)


@pytest.mark.parametrize("variant", [dict(force_sink=4, force_recent=64), dict(force_sink=0, force_recent=1),
                                     dict(force_sink=100, force_recent=0), dict(force_sink=4, force_recent=3000),
                                     dict(top_k=256, force_sink=4, force_recent=64),
                                     dict(top_k=5, force_sink=2000, force_recent=2000)])
def test_forced_positions(variant):
    dw, counts = _run(_ragged_config2(), **variant)
    # the variant adds something on these inputs (flat rows select a small share of a 3000-key context)
    assert any(c > reg for c, reg, _ in counts)


def test_forced_positions_with_exact_ties():
    gh = _harness()
    L = 9000
    wl = synth.config_1(L=L)
    wl.k[0][:, 0, :] = wl.k[0][0, 0, :]
    dw = gh.DeviceWorkload(wl, force_sink=4, force_recent=128)
    dw.index_all_keys()
    sc = dw.scores()[0]
    sel = dw.select()
    counts = gh.check_variant_selection(dw, sc, sel, force_sink=4, force_recent=128)
    c, reg, n = counts[0]
    assert c == reg + 128                                       # the first ~0.9 L positions, then the newest 128


def test_list_capacity_counts_forced_positions():
    gh = _harness()
    wl = synth.config_1(L=4096, n_needles=8)
    dw = gh.DeviceWorkload(wl, sel_stride=64, top_k=32, force_recent=64)
    dw.index_all_keys()
    sel = dw.select()
    assert int(sel["cnt"][0, 0]) > 64
    assert dw.status_code() == rb.RTP_ERR_CAPACITY


def test_chunk_and_block_forms_reject_the_variants():
    gh = _harness()
    wl = synth.config_3(L=512)
    pr = gh.PrefillRun(gh.DeviceWorkload(wl, top_k=16))
    pr.dw.index_all_keys()
    with pytest.raises(rb.RtpError) as e:
        pr.select_chunk(256, 256)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
