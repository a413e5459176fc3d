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
    sel_g = dw.select(general_path=True)
    gh.check_variant_selection(dw, sc, sel_g, rows=rows, **variant)
    sel = dw.select()
    counts = gh.check_variant_selection(dw, sc, sel, rows=rows, **variant)
    assert torch.equal(sel["cnt"], sel_g["cnt"]), "the two selection paths disagree"
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


# ---- mixed groups: retrieval and local query heads on one KV head (Section 3.2: the partition is over query heads) ----
def test_mixed_group_decode():
    """KV heads 0 and 1: two of the four query heads are retrieval heads, the other two attend locally."""
    gh = _harness()
    wl = synth.config_2(L=3000, batch=4, window=512, ret_per_group=2)
    assert wl.heads.ret_q_heads == [0, 1, 4, 5] and wl.heads.local_kv_heads == list(range(8))
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    qt = gh.check_queries(dw)
    sc = gh.check_scores(dw, qt)
    sel = dw.select()
    gh.check_selection(dw, sc, sel)
    # both calls write into ONE output: each must leave the other's heads alone
    out = torch.full((dw.R, 32, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((dw.R, 32), 7.0, dtype=torch.float32, device="cuda")
    rb.rtp_local_attn(dw.ctx, dw.params, dw.cache, dw.q, dw.row_seq, dw.row_pos, 0, 0, dw.R, out, lse, dw.workspace,
                      dw.status)
    torch.cuda.synchronize()
    o = out.float().cpu().numpy()
    assert np.all(o[:, wl.heads.ret_q_heads] == 7.0) and np.all(lse.cpu().numpy()[:, wl.heads.ret_q_heads] == 7.0)
    rb.rtp_sparse_attn_decode(dw.ctx, dw.params, dw.cache, dw.q, dw.row_seq, dw.row_pos, sel["idx"], sel["cnt"], out,
                              lse, dw.workspace, dw.status)
    torch.cuda.synchronize()
    o, l = out.float().cpu().numpy(), lse.cpu().numpy()
    gh.check_sparse_attention(dw, sel, o, l)
    gh.check_range_attention(dw, o, l, [0, 1, 5], "local")          # heads 2, 3, 6, 7 of the mixed groups and a plain one
    assert dw.status_code() == rb.RTP_OK


def test_mixed_group_decode_long_context_split_kv():
    """Long enough for the local call to split the window over several CTAs (the merge kernel must skip too)."""
    gh = _harness()
    wl = synth.config_2(L=20000, batch=2, window=8192, ret_per_group=1)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    out = torch.full((dw.R, 32, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((dw.R, 32), 7.0, dtype=torch.float32, device="cuda")
    rb.rtp_local_attn(dw.ctx, dw.params, dw.cache, dw.q, dw.row_seq, dw.row_pos, 0, 0, dw.R, out, lse, dw.workspace,
                      dw.status)
    torch.cuda.synchronize()
    o, l = out.float().cpu().numpy(), lse.cpu().numpy()
    assert wl.heads.ret_q_heads == [0, 4]
    assert np.all(o[:, [0, 4]] == 7.0) and np.all(l[:, [0, 4]] == 7.0)
    gh.check_range_attention(dw, o, l, [0, 1], "local")
    assert dw.status_code() == rb.RTP_OK


def test_mixed_group_prefill_lists_and_local():
    gh = _harness()
    wl = synth.config_3(L=768, window=128, ret_per_group=2)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    pr = gh.PrefillRun(dw)
    sel = pr.select_chunk(256, 512, with_lists=True)
    rows = [256, 500, 767]
    gh.check_chunk_selection(pr, 256, sel, rows)
    idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
    sets = {(m, i): idx[m - 256, i, : cnt[m - 256, i]] for m in rows for i in range(dw.n_ret)}
    o, l = pr.sparse_prefill(256, 512, sel, use_lists=True)
    gh.check_prefill_rows(pr, 256, o, l, rows, "sparse", None, sets)
    o, l = pr.local_prefill(256, 512)
    assert np.all(o[:, wl.heads.ret_q_heads] == 0)              # (the harness zero-fills the output)
    gh.check_prefill_rows(pr, 256, o, l, rows, "local", [0, 1, 4])
    # the threshold form needs index heads that cover whole groups
    with pytest.raises(rb.RtpError) as e:
        pr.sparse_prefill(256, 512, sel, use_lists=False)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
    assert dw.status_code() == rb.RTP_OK


def test_mixed_group_cannot_use_the_truncated_pool():
    wl = synth.config_2(L=300, batch=1, window=64, ret_per_group=2)
    params = rb.Params.from_workload(wl)
    dev = "cuda"
    z = lambda *shape: torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    bt = torch.zeros((1, 8), dtype=torch.int32, device=dev)
    lbt = torch.zeros((1, 4), dtype=torch.int32, device=dev)
    sl = torch.full((1,), 300, dtype=torch.int32, device=dev)
    cache = rb.make_cache(z(9, 1, 64, 128), z(9, 1, 64, 128), z(9, 2, 64, 16), bt, sl, k_local_pages=z(5, 8, 64, 128),
                          v_local_pages=z(5, 8, 64, 128), local_block_table=lbt, sink_pages=1)
    q = z(1, 32, 128)
    out = z(1, 32, 128)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rs = torch.zeros(1, dtype=torch.int32, device=dev)
    rp = torch.full((1,), 299, dtype=torch.int32, device=dev)
    with pytest.raises(rb.RtpError) as e:
        rb.rtp_local_attn(rb.Context(), params, cache, q, rs, rp, 0, 0, 1, out,
                          torch.zeros((1, 32), dtype=torch.float32, device=dev), ws, st)
    assert e.value.code == rb.RTP_ERR_INVALID
