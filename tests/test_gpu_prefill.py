"""GPU parity of the prefill path (S0-S4 per chunk, S6, S7, S9) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _gh():
    from tests import gpu_harness as gh
    return gh


def _sample_rows(q_start, C, rng, extra=()):
    rows = {q_start, q_start + C - 1, q_start + C // 2}
    rows |= set(int(x) for x in rng.integers(q_start, q_start + C, 5))
    rows |= set(int(x) for x in extra if q_start <= x < q_start + C)
    return sorted(rows)


def _prep(wl):
    gh = _gh()
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    return gh, dw, gh.PrefillRun(dw)


@pytest.mark.parametrize("L,chunk", [(1000, 600), (2048, 1024), (130, 130)])
def test_dense_and_local_prefill(L, chunk):
    wl = synth.config_3(L=L, window=200)
    gh, dw, pr = _prep(wl)
    rng = np.random.default_rng(L)
    for q_start in range(0, L, chunk):
        C = min(chunk, L - q_start)
        rows = _sample_rows(q_start, C, rng, extra=(3, 4, 63, 64, 199, 200, 201, 263, 264))
        out, lse = pr.dense_prefill(q_start, C, kv_heads=[0, 5])
        gh.check_prefill_rows(pr, q_start, out, lse, rows, "dense", [0, 5])
        out, lse = pr.local_prefill(q_start, C)
        gh.check_prefill_rows(pr, q_start, out, lse, rows, "local", wl.heads.local_kv_heads[:2])
        assert np.all(out[:, wl.heads.ret_q_heads] == 0)        # retrieval slots untouched by the local call
    assert dw.status_code() == rb.RTP_OK


def test_config3_reduced_select_and_sparse_prefill():
    wl = synth.config_3(L=3000, window=512)
    gh, dw, pr = _prep(wl)
    rng = np.random.default_rng(3)
    all_fracs = []
    for q_start, C in [(0, 1024), (1024, 1024), (2048, 952)]:
        rows = _sample_rows(q_start, C, rng)
        sel = pr.select_chunk(q_start, C, with_lists=True)
        sc, fracs = gh.check_chunk_selection(pr, q_start, sel, rows)
        all_fracs += fracs
        idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
        sets = {(m, i): idx[m - q_start, i, : cnt[m - q_start, i]] for m in rows for i in range(dw.n_ret)}
        out_t, lse_t = pr.sparse_prefill(q_start, C, sel, use_lists=False)
        gh.check_prefill_rows(pr, q_start, out_t, lse_t, rows, "sparse", None, sets)
        out_l, lse_l = pr.sparse_prefill(q_start, C, sel, use_lists=True)
        gh.check_prefill_rows(pr, q_start, out_l, lse_l, rows, "sparse", None, sets)
        h = wl.heads.ret_q_heads
        # both routes agree on every row (each is within 2e-2 of the exact result)
        assert np.abs(out_t[:, h] - out_l[:, h]).max() <= 4e-2
        # thresholds-only call gives the same thresholds
        sel2 = pr.select_chunk(q_start, C, with_lists=False)
        assert torch.equal(sel2["cnt"], sel["cnt"]) and torch.equal(sel2["tie"], sel["tie"])
        assert torch.equal(sel2["thr"], sel["thr"])
    assert dw.status_code() == rb.RTP_OK
    assert 0.005 <= np.mean(all_fracs) <= 0.6


@pytest.mark.parametrize("amp,top_p", [(3, 0.9), (1, 0.5), (6, 0.99)])
def test_select_scores_on_bin_boundaries_and_heavy_ties(amp, top_p):
    """Integer-valued index features with temperature 1/8: scores are multiples of 1/8, so half of them sit exactly between
    two of the selection kernel's quarter-wide bins, and every score value is shared by many keys."""
    wl = synth.config_grid_ties(L=3000, amp=amp, top_p=top_p)
    gh, dw, pr = _prep(wl)
    rng = np.random.default_rng(amp)
    for q_start, C in [(0, 1024), (1024, 1024), (2048, 952)]:
        rows = _sample_rows(q_start, C, rng, extra=(1, 2, 5, 63, 64, 65))
        sel = pr.select_chunk(q_start, C, with_lists=True)
        sc, _ = gh.check_chunk_selection(pr, q_start, sel, rows)
        assert np.all(sc[np.isfinite(sc)] * 8 == np.round(sc[np.isfinite(sc)] * 8))      # the input does what it says
        sel2 = pr.select_chunk(q_start, C, with_lists=False)
        assert torch.equal(sel2["cnt"], sel["cnt"]) and torch.equal(sel2["tie"], sel["tie"])
        assert torch.equal(sel2["thr"], sel["thr"])
        idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
        sets = {(m, i): idx[m - q_start, i, : cnt[m - q_start, i]] for m in rows for i in range(dw.n_ret)}
        out_t, lse_t = pr.sparse_prefill(q_start, C, sel, use_lists=False)
        gh.check_prefill_rows(pr, q_start, out_t, lse_t, rows, "sparse", None, sets)
    assert dw.status_code() == rb.RTP_OK


@pytest.mark.parametrize("n_q,n_kv", [(16, 2), (4, 2), (2, 2)])
def test_other_group_sizes(n_q, n_kv):
    """G = 8, 2 and 1 query heads per KV head: 16, 64 and 128 positions per CTA tile in the chunk kernels."""
    wl = synth.config_3(L=1400, n_q_heads=n_q, n_kv_heads=n_kv, ret_kv_heads=(0,), window=300)
    gh, dw, pr = _prep(wl)
    rng = np.random.default_rng(n_q)
    for q_start, C in [(0, 700), (700, 700)]:
        rows = _sample_rows(q_start, C, rng, extra=(15, 16, 17, 63, 64, 127, 128, 129))
        sel = pr.select_chunk(q_start, C, with_lists=True)
        gh.check_chunk_selection(pr, q_start, sel, rows)
        idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
        sets = {(m, i): idx[m - q_start, i, : cnt[m - q_start, i]] for m in rows for i in range(dw.n_ret)}
        out, lse = pr.sparse_prefill(q_start, C, sel, use_lists=False)
        gh.check_prefill_rows(pr, q_start, out, lse, rows, "sparse", None, sets)
        out, lse = pr.local_prefill(q_start, C)
        gh.check_prefill_rows(pr, q_start, out, lse, rows, "local", wl.heads.local_kv_heads[:1])
        out, lse = pr.dense_prefill(q_start, C, kv_heads=[1])
        gh.check_prefill_rows(pr, q_start, out, lse, rows, "dense", [1])
    assert dw.status_code() == rb.RTP_OK


def test_config4_reduced_needle_rows():
    wl = synth.config_4(L=4096, n_needles=32)
    gh, dw, pr = _prep(wl)
    qrows = wl.notes["needle_query_row"]
    sel = pr.select_chunk(0, 4096, with_lists=True, stride=4096)
    rows = sorted(set(int(x) for x in qrows[:6]) | {0, 1, 4095, 2000})
    sc, fracs = gh.check_chunk_selection(pr, 0, sel, rows)
    idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
    # a needle row keeps few keys and its planted key is among them
    hits = 0
    for kpos, r in zip(wl.notes["needle_key_pos"], qrows):
        if kpos in set(idx[r, 0, : cnt[r, 0]].tolist()):
            hits += 1
    assert hits >= 0.9 * len(qrows)
    sets = {(m, i): idx[m, i, : cnt[m, i]] for m in rows for i in range(dw.n_ret)}
    out, lse = pr.sparse_prefill(0, 4096, sel, use_lists=False)
    gh.check_prefill_rows(pr, 0, out, lse, rows, "sparse", None, sets)
    assert dw.status_code() == rb.RTP_OK


def test_chunk_and_row_selection_agree_and_decode_equals_last_prefill_row():
    wl = synth.config_3(L=1500, window=256)
    gh, dw, pr = _prep(wl)
    sel = pr.select_chunk(1000, 500, with_lists=True)
    rows = [1000, 1234, 1499]
    sc, _ = gh.check_chunk_selection(pr, 1000, sel, rows)
    # the same rows through the explicit-row (decode) entry points
    q = dw.q[torch.tensor(rows, device="cuda")].contiguous()
    R = len(rows)
    row_seq, row_pos = gh.dev_i32(np.zeros(R)), gh.dev_i32(rows)
    idx = torch.full((R, dw.n_ret, 1500), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros((R, dw.n_ret), dtype=torch.int32, device="cuda")
    mass = torch.zeros((R, dw.n_ret), device="cuda")
    thr = torch.zeros((R, dw.n_ret), device="cuda")
    tie = torch.zeros((R, dw.n_ret), dtype=torch.int32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(dw.params, R, 1500), dtype=torch.uint8, device="cuda")
    rb.rtp_topp_select(dw.ctx, dw.params, dw.cache, q, dw.w_q, row_seq, row_pos, 0, 0, R, idx, cnt, mass, thr, tie,
                       dw.status, ws)
    out_d = torch.zeros((R, 32, 128), dtype=torch.bfloat16, device="cuda")
    rb.rtp_sparse_attn_decode(dw.ctx, dw.params, dw.cache, q, row_seq, row_pos, idx, cnt, out_d, None, ws, dw.status)
    torch.cuda.synchronize()
    c_chunk = sel["cnt"].cpu().numpy()
    for k, m in enumerate(rows):
        for i in range(dw.n_ret):
            a = set(idx[k, i, : int(cnt[k, i])].cpu().numpy().tolist())
            b = set(sel["idx"][m - 1000, i, : c_chunk[m - 1000, i]].cpu().numpy().tolist())
            assert len(a ^ b) <= 2                                # only band-edge tokens may differ
    out_p, _ = pr.sparse_prefill(1000, 500, sel, use_lists=False)
    h = wl.heads.ret_q_heads
    od = out_d.float().cpu().numpy()
    for k, m in enumerate(rows):
        assert np.abs(od[k][h] - out_p[m - 1000][h]).max() <= 2e-2
    # local / dense: decode row == prefill row
    lo_p, _ = pr.local_prefill(1000, 500)
    out_l = torch.zeros((R, 32, 128), dtype=torch.bfloat16, device="cuda")
    rb.rtp_local_attn(dw.ctx, dw.params, dw.cache, q, row_seq, row_pos, 0, 0, R, out_l, None, ws, dw.status)
    torch.cuda.synchronize()
    ol = out_l.float().cpu().numpy()
    lh = [kv * 4 + j for kv in wl.heads.local_kv_heads for j in range(4)]
    for k, m in enumerate(rows):
        assert np.abs(ol[k][lh] - lo_p[m - 1000][lh]).max() <= 2e-2
    assert dw.status_code() == rb.RTP_OK


def test_prefill_independent_of_chunk_size():
    wl = synth.config_3(L=1024, window=300)
    gh, dw, pr = _prep(wl)
    whole_l, _ = pr.local_prefill(0, 1024)
    whole_sel = pr.select_chunk(0, 1024, with_lists=False)
    whole_s, _ = pr.sparse_prefill(0, 1024, whole_sel, use_lists=False)
    parts_l, parts_s, cnts = [], [], []
    for q_start, C in [(0, 100), (100, 412), (512, 512)]:
        parts_l.append(pr.local_prefill(q_start, C)[0])
        sel = pr.select_chunk(q_start, C, with_lists=False)
        cnts.append(sel["cnt"].cpu().numpy())
        parts_s.append(pr.sparse_prefill(q_start, C, sel, use_lists=False)[0])
    assert np.abs(np.concatenate(parts_l) - whole_l).max() <= 1e-2
    assert np.abs(np.concatenate(parts_s) - whole_s).max() <= 2e-2
    assert np.abs(np.concatenate(cnts) - whole_sel["cnt"].cpu().numpy()).max() <= 2


def test_top_p_one_prefill_equals_dense():
    wl = synth.config_3(L=700, window=128)
    wl.top_p = 1.0
    gh, dw, pr = _prep(wl)
    sel = pr.select_chunk(0, 700, with_lists=False)
    assert np.array_equal(sel["cnt"].cpu().numpy()[:, 0], np.arange(1, 701))
    out_s, lse_s = pr.sparse_prefill(0, 700, sel, use_lists=False)
    out_d, lse_d = pr.dense_prefill(0, 700, kv_heads=wl.heads.ret_kv_heads)
    h = wl.heads.ret_q_heads
    assert np.abs(out_s[:, h] - out_d[:, h]).max() <= 3e-2        # two kernels, each bf16-rounded
    np.testing.assert_allclose(lse_s[:, h], lse_d[:, h], rtol=1e-4, atol=1e-4)


def test_equal_scores_in_a_chunk_take_lowest_positions():
    wl = synth.config_3(L=600, window=128)
    wl.k[0][:, 0, :] = wl.k[0][0, 0, :]                        # identical keys on KV head 0 -> all scores tie
    gh, dw, pr = _prep(wl)
    sel = pr.select_chunk(0, 600, with_lists=True)
    cnt, tie, idx = sel["cnt"].cpu().numpy(), sel["tie"].cpu().numpy(), sel["idx"].cpu().numpy()
    for m in [0, 1, 9, 10, 99, 599]:
        want = int(np.ceil(0.9 * (m + 1) - 1e-9))
        for i in range(4):                                     # heads of KV head 0
            c = int(cnt[m, i])
            assert want <= c <= want + 1
            assert sorted(idx[m, i, :c].tolist()) == list(range(c))
            assert tie[m, i] >= c - 1
    rows = [5, 300, 599]
    gh.check_chunk_selection(pr, 0, sel, rows)
    assert dw.status_code() == rb.RTP_OK
