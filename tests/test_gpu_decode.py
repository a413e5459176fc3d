"""GPU parity of the decode path (S0-S5, S7-S9) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as gh
    return gh


def _run_decode(wl, sel_stride=None, check_rows=None, dense_heads=(0,)):
    gh = _harness()
    dw = gh.DeviceWorkload(wl, sel_stride=sel_stride)
    dw.index_all_keys()
    gh.check_index_keys(dw)
    qt = gh.check_queries(dw)
    sc = gh.check_scores(dw, qt, rows=check_rows)
    # the decode selection has two implementations (one CTA per (row, head) for short contexts, several kernels over
    # stored scores otherwise): both are checked, and they must agree exactly
    sel_g = dw.select(general_path=True)
    gh.check_selection(dw, sc, sel_g, rows=check_rows)
    sel = dw.select()
    stats = gh.check_selection(dw, sc, sel, rows=check_rows)
    for k in ("cnt", "thr", "tie"):
        assert torch.equal(sel[k], sel_g[k]), f"the two selection paths disagree on {k}"
    assert torch.equal(torch.sort(sel["idx"], dim=-1).values, torch.sort(sel_g["idx"], dim=-1).values)
    out, lse = dw.sparse_decode()
    gh.check_sparse_attention(dw, sel, out, lse, rows=check_rows)
    if wl.heads.local_kv_heads:
        lo, ll = dw.local_decode()
        gh.check_range_attention(dw, lo, ll, wl.heads.local_kv_heads[:2], "local", rows=check_rows)
        # slots of retrieval heads are not touched by the local call
        assert np.all(lo[:, wl.heads.ret_q_heads] == 0)
    do, dl = dw.dense_decode(list(dense_heads))
    gh.check_range_attention(dw, do, dl, list(dense_heads), "dense", rows=check_rows)
    assert dw.status_code() == rb.RTP_OK
    return dw, stats


def test_config1_single_decode_with_needles():
    wl = synth.config_1()
    dw, stats = _run_decode(wl)
    c, k_star, n = stats[0]
    assert n == 4096 and 1 <= c <= 16
    got = set(dw.sel["idx"][0, 0, :c].cpu().numpy().tolist())
    assert got <= set(wl.notes["needles"].tolist())          # only planted keys are selected


@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 130, 1000])
def test_config1_ragged_lengths(L):
    _run_decode(synth.config_1(L=L, n_needles=min(8, max(1, L // 4))))


def test_config2_reduced_with_ragged_batch():
    wl = synth.config_2(L=3000, batch=4, window=512)
    # make the batch ragged: shorten every sequence differently
    for b, cut in enumerate([0, 517, 1, 2049]):
        L = 3000 - cut
        wl.k[b], wl.v[b] = wl.k[b][:L], wl.v[b][:L]
        wl.seq_lens[b] = L
        wl.row_pos[b] = L - 1
    _run_decode(wl, dense_heads=(0, 5))


def test_group_of_eight_query_heads_per_kv_head():
    """G = 8: eight retrieval heads share one index head (the selection kernels' path for more than four heads)."""
    wl = synth.config_2(L=2600, batch=2, n_q_heads=16, n_kv_heads=2, ret_kv_heads=(0,), window=300)
    _run_decode(wl, dense_heads=(0,))


def test_config2_full_size():
    wl = synth.config_2()
    dw, stats = _run_decode(wl, dense_heads=(1,))
    peaked = [c for (c, k, n) in stats[: 4 * 8]]
    flat = [c / n for (c, k, n) in stats[4 * 8:]]
    assert np.median(peaked) <= 80                            # mostly the planted keys
    assert 0.05 <= np.mean(flat) <= 0.35                      # iid keys: a two-digit percentage


def test_config5_point_128k():
    wl = synth.config_5(L=131072, batch=1, top_p=0.9, frac=0.05)
    dw, stats = _run_decode(wl, sel_stride=40000, dense_heads=(7,))
    fr = [c / n for (c, k, n) in stats]
    assert 0.01 <= np.mean(fr) <= 0.12


@pytest.mark.parametrize("top_p,frac,batch,L", [(0.8, 0.2, 2, 20000), (0.99, 0.01, 3, 30000), (0.9, 0.001, 16, 9000),
                                                 (0.99, 0.2, 1, 70000)])
def test_config5_sweep_corners(top_p, frac, batch, L):
    """Corners of the long-context sweep at sizes the oracle finishes quickly: top-p 0.8 .. 0.99, selected fractions
    0.1 % .. 20 %, batch 1 .. 16 (the 20 % / 70K point needs a key level and more than 4096 candidates per level-1 bin)."""
    wl = synth.config_5(L=L, batch=batch, top_p=top_p, frac=frac)
    dw, stats = _run_decode(wl, sel_stride=int(min(L, max(4096, 4 * frac * L))), dense_heads=(3,))
    fr = np.array([c / n for (c, k, n) in stats])
    assert 0.2 * frac <= fr.mean() <= 4.0 * frac


def test_top_p_one_selects_everything_and_equals_dense():
    gh = _harness()
    wl = synth.config_2(L=700, batch=2, window=512)
    wl.top_p = 1.0
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    sel = dw.select()
    assert np.all(sel["cnt"].cpu().numpy() == 700)
    out, lse = dw.sparse_decode()
    do, dl = dw.dense_decode(wl.heads.ret_kv_heads)
    h = wl.heads.ret_q_heads
    assert np.abs(out[:, h] - do[:, h]).max() <= 2e-2
    gh.check_range_attention(dw, out, lse, wl.heads.ret_kv_heads, "dense")


@pytest.mark.parametrize("L", [100, 5000, 9000])
def test_equal_scores_take_lowest_positions(L):
    """All index keys equal -> all scores tie; the canonical set is the first ceil(p L) positions.
    L > 4096 exercises the exact-tie path that cannot buffer all candidates."""
    gh = _harness()
    wl = synth.config_1(L=L)
    wl.k[0][:, 0, :] = wl.k[0][0, 0, :]                        # identical keys
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    sc = dw.scores()[0]
    assert np.all(sc[0, 0, :L] == sc[0, 0, 0])
    sel = dw.select()
    c = int(sel["cnt"][0, 0])
    want = int(np.ceil(0.9 * L - 1e-9))
    assert want <= c <= want + int(2e-4 * L) + 1
    assert sorted(sel["idx"][0, 0, :c].cpu().numpy().tolist()) == list(range(c))
    assert int(sel["tie"][0, 0]) == c - 1
    gh.check_selection(dw, sc, sel)


def test_dense_cluster_of_near_equal_scores():
    """12000 keys that differ from one needle key by single bf16 mantissa bits: their scores crowd into one level-1
    bin (far more than the 4096 candidates the exact finish takes), many tie exactly, and the cut falls among them:
    several key levels, the one-CTA tail pass and the tie rule all have to agree with the oracle."""
    wl = synth.config_1(L=20000, n_needles=4)
    K = wl.k[0]                                                 # bf16 bit patterns, [L, 1, 128]
    rng = np.random.default_rng(7)
    base = K[int(wl.notes["needles"][0]), 0].copy()
    for n in range(3000, 15000):
        k = base.copy()
        dims = rng.integers(0, 128, size=3)
        k[dims] ^= np.uint16(1)                                # one mantissa ulp in three dimensions
        K[n, 0] = k
    dw, stats = _run_decode(wl, sel_stride=20000)
    c, k_star, n = stats[0]
    assert 8000 <= c <= 12100                                   # about 90 % of the cluster carries 90 % of the mass


def test_dense_cluster_in_a_short_context():
    """The same kind of cluster in a context short enough for the one-CTA selection: 8000 near-equal scores, twice the
    candidates its finish takes, so its key levels and its tie rule are exercised (and compared with the general path)."""
    wl = synth.config_1(L=12000, n_needles=4)
    K = wl.k[0]
    rng = np.random.default_rng(11)
    base = K[int(wl.notes["needles"][0]), 0].copy()
    for n in range(2000, 10000):
        k = base.copy()
        dims = rng.integers(0, 128, size=3)
        k[dims] ^= np.uint16(1)
        K[n, 0] = k
    dw, stats = _run_decode(wl, sel_stride=12000)
    c, k_star, n = stats[0]
    assert 5000 <= c <= 8100


@pytest.mark.parametrize("general", [False, True])
def test_counts_only_selection_matches_the_lists(general):
    gh = _harness()
    wl = synth.config_2(L=3000, batch=4, window=512)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    a = dw.select(general_path=general)
    a = {k: (v.clone() if v is not None else None) for k, v in a.items()}
    b = dw.select(with_lists=False, general_path=general)
    for k in ("cnt", "mass", "thr", "tie"):
        assert torch.equal(a[k], b[k]), k
    assert dw.status_code() == rb.RTP_OK


def test_window_larger_than_context_equals_dense():
    gh = _harness()
    wl = synth.config_2(L=900, batch=2, window=4096)
    dw = gh.DeviceWorkload(wl)
    lo, ll = dw.local_decode()
    do, dl = dw.dense_decode(wl.heads.local_kv_heads)
    h = [kv * 4 + j for kv in wl.heads.local_kv_heads for j in range(4)]
    assert np.array_equal(lo[:, h], do[:, h])
    np.testing.assert_allclose(ll[:, h], dl[:, h], rtol=1e-6)


def test_list_overflow_reports_capacity_and_true_count():
    gh = _harness()
    wl = synth.config_5(L=8192, batch=1, frac=0.2)
    dw = gh.DeviceWorkload(wl, sel_stride=64)
    dw.index_all_keys()
    sel = dw.select()
    cnt = sel["cnt"].cpu().numpy()
    assert cnt.max() > 64
    assert dw.status_code() == rb.RTP_ERR_CAPACITY
    idx = sel["idx"].cpu().numpy()
    assert np.all(idx >= 0) and np.all(idx < 8192)             # the first 64 ids of every row are valid


def test_row_beyond_sequence_is_reported_not_trapped():
    gh = _harness()
    wl = synth.config_1(L=256)
    wl.row_pos[0] = 300
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    dw.select()
    assert dw.status_code() == rb.RTP_ERR_INVALID
    assert int(dw.sel["cnt"][0, 0]) <= 256


def test_host_side_argument_errors():
    gh = _harness()
    wl = synth.config_1(L=256)
    dw = gh.DeviceWorkload(wl)
    with pytest.raises(rb.RtpError) as e:
        rb.rtp_topp_select(dw.ctx, dw.params, dw.cache, dw.q, dw.w_q, dw.row_seq, None, 0, 0, 1, None,
                           torch.zeros(1, dtype=torch.int32, device="cuda"), None, None, None, dw.status, dw.workspace)
    assert e.value.code == rb.RTP_ERR_INVALID
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(rb.RtpError) as e:
        rb.rtp_topp_select(dw.ctx, dw.params, dw.cache, dw.q, dw.w_q, dw.row_seq, dw.row_pos, 0, 0, 1, None,
                           torch.zeros(1, dtype=torch.int32, device="cuda"), None, None, None, dw.status, small)
    assert e.value.code == rb.RTP_ERR_CAPACITY
    bad = rb.Params.from_workload(wl, top_p=0.0)
    with pytest.raises(rb.RtpError):
        rb.rtp_index_queries(dw.ctx, bad, dw.q, dw.w_q, torch.empty((1, 1, 16), dtype=torch.bfloat16, device="cuda"))


def test_kv_append_writes_pages_bit_exactly():
    gh = _harness()
    wl = synth.config_2(L=333, batch=3, window=128)
    dw = gh.DeviceWorkload(wl)
    want_k, want_v = dw.k_pages.clone(), dw.v_pages.clone()
    dw.k_pages.zero_()
    dw.v_pages.zero_()
    for b in range(3):
        k = gh.dev_bf16(wl.k[b])
        v = gh.dev_bf16(wl.v[b])
        seq = torch.full((333,), b, dtype=torch.int32, device="cuda")
        pos = torch.arange(333, dtype=torch.int32, device="cuda")
        rb.rtp_kv_append(dw.ctx, dw.params, dw.cache, k, v, seq, pos, dw.status)
    torch.cuda.synchronize()
    assert torch.equal(dw.k_pages.view(torch.int16), want_k.view(torch.int16))
    assert torch.equal(dw.v_pages.view(torch.int16), want_v.view(torch.int16))
    assert dw.status_code() == rb.RTP_OK
    # a token outside the block table is skipped and reported
    rb.rtp_kv_append(dw.ctx, dw.params, dw.cache, gh.dev_bf16(wl.k[0][:1]), gh.dev_bf16(wl.v[0][:1]),
                     torch.tensor([7], dtype=torch.int32, device="cuda"),
                     torch.tensor([0], dtype=torch.int32, device="cuda"), dw.status)
    assert dw.status_code() == rb.RTP_ERR_INVALID
