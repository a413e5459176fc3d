"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the CUDA path runs
the whole workload (or, at one million tokens, the chunks that hold the sampled rows), the oracle checks
sampled rows one by one.

Stage-wise checks (teacher forced): GPU-written index keys and projected queries feed the oracle's scoring;
the selection is judged on the GPU's own materialised scores; attention on the GPU's own set.
End-to-end checks: the oracle runs the whole row from the raw bf16 inputs (its own projections, scores and
set); the GPU's set may differ from the oracle's only in tokens whose oracle score lies within the score
tolerance of the oracle's threshold, or inside the 1e-4 mass band."""
import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import binding as rb
from tests.set_checks import e2e_set_check as _e2e_set_check

pytestmark = pytest.mark.gpu


def _np16(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _gpu_scores(path, data, rows, L):
    """Materialised GPU scores and projected queries of the given positions (explicit-row entry points)."""
    R = len(rows)
    qrows = data.q[torch.tensor(rows, device="cuda")].contiguous()
    qt = torch.empty((R, path.n_ret, 16), dtype=torch.bfloat16, device="cuda")
    rb.rtp_index_queries(path.ctx, path.params, qrows, data.w_q, qt)
    sc = torch.full((R, path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, R, L), dtype=torch.uint8, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, qrows, data.w_q,
                       torch.zeros(R, dtype=torch.int32, device="cuda"),
                       torch.tensor(rows, dtype=torch.int32, device="cuda"), sc, None, None, ws, path.status)
    torch.cuda.synchronize()
    return sc.cpu().numpy(), _np16(qt), _np16(qrows)


def _score_tol(want_s, qt_u16, kt_u16, scale):
    qn = np.linalg.norm(orc.bf16_to_f64(qt_u16))
    kn = np.linalg.norm(orc.bf16_to_f64(kt_u16), axis=-1)
    return 1e-3 * np.abs(want_s) + 1e-5 * scale * qn * kn



def check_prefill_rows_stagewise(data, path, rows, L, sel, out_h, lse_h, local_heads=2, e2e_rows=()):
    """sel: dict row -> (thr, tie, cnt, mass) arrays [n_ret]; out_h / lse_h: dict row -> arrays [Hq, ...]."""
    heads, g = data.heads, data.heads.group
    ik = _np16(path.ikey_pages[data.block_table[0].long()])               # [pages, nih, 64, 16]
    kt = np.transpose(ik, (0, 2, 1, 3)).reshape(-1, heads.n_index_heads, 16)[:L]
    sc, qt, qh = _gpu_scores(path, data, rows, L)
    w_q, w_k = _np16(data.w_q), _np16(data.w_k)
    kv, kt_oracle, fr = {}, {}, []
    for k, m in enumerate(rows):
        thr_r, tie_r, cnt_r, mass_r = sel[m]
        for i, h in enumerate(heads.ret_q_heads):
            kh, j = h // g, heads.q_head_to_index_head[i]
            if kh not in kv:
                kv[kh] = data.logical_kv(0, kh)
            s = sc[k, i, : m + 1]
            want_s = orc.index_scores(qt[k, i], kt[: m + 1, j], data.score_scale)
            assert np.all(np.abs(s - want_s) <= _score_tol(want_s, qt[k, i], kt[: m + 1, j], data.score_scale)), f"row {m} head {i}"
            member = (s > thr_r[i]) | ((s == thr_r[i]) & (np.arange(m + 1) <= tie_r[i]))
            got = set(np.nonzero(member)[0].tolist())
            assert len(got) == int(cnt_r[i]), f"row {m} head {i}: rule gives {len(got)}, count {int(cnt_r[i])}"
            mand, forb = orc.classify_against_band(s, data.top_p)
            assert mand <= got and not (forb & got), f"row {m} head {i}"
            tm = orc.set_mass(s, got)
            assert tm >= data.top_p or len(got) == m + 1
            assert abs(tm - mass_r[i]) <= 1e-4
            want, wlse = orc.attention_over_set(qh[k, h], kv[kh][0], kv[kh][1], sorted(got), data.sm_scale)
            assert np.abs(out_h[m][h] - want).max() <= 2e-2, f"sparse row {m} head {h}"
            assert abs(lse_h[m][h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
            fr.append(len(got) / (m + 1))
            if m in e2e_rows:
                # end to end from the raw inputs: the oracle projects, scores, selects and attends on its own
                if j not in kt_oracle:
                    kt_oracle[j] = orc.index_project(kv[heads.index_head_kv[j]][0], w_k[j])
                ref = orc.retrieval_row(qh[k, h], qh[k, h], w_q[i], kt_oracle[j], kv[kh][0], kv[kh][1], m, data.top_p,
                                        data.score_scale, data.sm_scale)
                so = ref["scores"]
                qf, kf = orc.bf16_to_f64(ref["qt"]), orc.bf16_to_f64(kt_oracle[j][: m + 1])
                # tolerance on a score: 1e-3 relative, plus one bf16 step on every stored projection component
                tol = 1e-3 * np.abs(so) + 2.0 ** -7 * data.score_scale * (np.abs(kf) @ np.abs(qf))
                eps = _e2e_set_check(so, s, got, data.top_p, tol, f"e2e row {m} head {i}")
                assert orc.set_mass(so, got) >= data.top_p - eps or len(got) == m + 1
                if got == set(ref["ids"].tolist()):
                    assert np.abs(out_h[m][h] - ref["out"]).max() <= 2e-2, f"e2e output row {m} head {h}"
        for kh in heads.local_kv_heads[:local_heads]:
            if kh not in kv:
                kv[kh] = data.logical_kv(0, kh)
            for jj in range(g):
                h = kh * g + jj
                want, wlse = orc.local_row(qh[k, h], kv[kh][0], kv[kh][1], m, heads.n_sink, heads.window, data.sm_scale)
                assert np.abs(out_h[m][h] - want).max() <= 2e-2, f"local row {m} head {h}"
                assert abs(lse_h[m][h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
    return fr


def test_prefill_128k_sampled_rows():
    from paper_2605_16928_b200 import pipeline, synth_device
    L, chunk = 131072, 8192
    data = synth_device.config_3_device(L=L)
    path = pipeline.PrefillPath(data, chunk)
    k_pre = data.k_pre_rows(0, 0, L)
    out = torch.zeros((L, 32, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((L, 32), dtype=torch.float32, device="cuda")
    thr = torch.zeros((L, path.n_ret), dtype=torch.float32, device="cuda")
    tie = torch.zeros((L, path.n_ret), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((L, path.n_ret), dtype=torch.int32, device="cuda")
    mass = torch.zeros((L, path.n_ret), dtype=torch.float32, device="cuda")
    for (s, C) in path.chunks():
        path.run_chunk(s, C, data.q[s:s + C], k_pre[s:s + C], out[s:s + C], lse[s:s + C])
        thr[s:s + C], tie[s:s + C] = path.sel_thr[:C], path.sel_tie[:C]
        cnt[s:s + C], mass[s:s + C] = path.sel_cnt[:C], path.sel_mass[:C]
    torch.cuda.synchronize()
    assert path.status_code() == rb.RTP_OK
    rng = np.random.default_rng(1)
    # first and last row of every chunk, a few rows around page and tile boundaries, 64 random rows
    rows = {0, 1, 63, 64, 127, 128}
    for (s, C) in path.chunks():
        rows |= {s, s + C - 1}
    rows |= set(map(int, rng.integers(0, L, 64)))
    rows = sorted(rows)
    idx_t = torch.tensor(rows, device="cuda")
    thr_h, tie_h, cnt_h, mass_h = (x[idx_t].cpu().numpy() for x in (thr, tie, cnt, mass))
    out_r, lse_r = out[idx_t].float().cpu().numpy(), lse[idx_t].cpu().numpy()
    sel = {m: (thr_h[k], tie_h[k], cnt_h[k], mass_h[k]) for k, m in enumerate(rows)}
    fr = check_prefill_rows_stagewise(data, path, rows, L, sel, {m: out_r[k] for k, m in enumerate(rows)},
                                      {m: lse_r[k] for k, m in enumerate(rows)},
                                      e2e_rows=set(rows[::12]))
    assert 0.002 <= float(np.mean(fr)) <= 0.6


def test_prefill_1m_config4_sampled_rows():
    """Config 4 (one million tokens, chunk 16K, one retrieval KV head, planted needles): only the chunks that hold the
    sampled rows are run; K/V and the index keys of the whole sequence are resident."""
    from paper_2605_16928_b200 import pipeline, synth_device
    L, chunk = 1048576, 16384
    data = synth_device.config_4_device(L=L)
    path = pipeline.PrefillPath(data, chunk)
    for s in range(0, L, 131072):                       # index keys of the whole sequence
        path.index_keys_range(0, s, min(L, s + 131072))
    kpos, qrow = data.notes["needle_key_pos"], data.notes["needle_query_row"]
    rng = np.random.default_rng(4)
    pick = rng.choice(len(qrow), 8, replace=False)
    rows = sorted({0, L - 1, *map(int, qrow[pick]), *map(int, rng.integers(0, L, 8))})
    needle_of = {int(qrow[i]): int(kpos[i]) for i in pick}
    sel, out_h, lse_h = {}, {}, {}
    out = torch.zeros((chunk, 32, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((chunk, 32), dtype=torch.float32, device="cuda")
    for s in sorted({(m // chunk) * chunk for m in rows}):
        C = min(chunk, L - s)
        path.run_chunk(s, C, data.q[s:s + C], data.k_pre_rows(0, s, s + C), out[:C], lse[:C])
        torch.cuda.synchronize()
        for m in rows:
            if s <= m < s + C:
                r = m - s
                sel[m] = tuple(x[r].cpu().numpy() for x in (path.sel_thr, path.sel_tie, path.sel_cnt, path.sel_mass))
                out_h[m], lse_h[m] = out[r].float().cpu().numpy(), lse[r].cpu().numpy()
    assert path.status_code() == rb.RTP_OK
    fr = check_prefill_rows_stagewise(data, path, rows, L, sel, out_h, lse_h, local_heads=1, e2e_rows={rows[1], rows[-1]})
    assert 0.0 < float(np.mean(fr)) <= 0.3
    # a needle row keeps few keys, and its planted key is among them
    sc, _, _ = _gpu_scores(path, data, sorted(needle_of), L)
    for k, m in enumerate(sorted(needle_of)):
        thr_r, tie_r, cnt_r, _ = sel[m]
        for i in range(path.n_ret):
            s_n = sc[k, i, needle_of[m]]
            assert s_n > thr_r[i] or (s_n == thr_r[i] and needle_of[m] <= tie_r[i]), f"needle row {m} head {i}"
            assert int(cnt_r[i]) <= 64, f"needle row {m} head {i} keeps {int(cnt_r[i])} keys"


def _decode_point(L, B, top_p, frac, window, seqs, peaked_half=False, name="c5_decode_sweep", e2e=True, **path_kw):
    from paper_2605_16928_b200 import pipeline, synth_device
    data = synth_device.decode_device(L, B, top_p, frac, window, peaked_half=peaked_half, name=name)
    path = pipeline.DecodePath(data, sel_stride=int(min(L, max(16384, 4 * frac * L))), **path_kw)
    path.build_index_cache()
    k_new = torch.stack([data.k_pre_rows(b, L - 1, L)[0] for b in range(B)]).contiguous()
    path.step(data.q, k_new)
    torch.cuda.synchronize()
    assert path.status_code() == rb.RTP_OK
    heads, g = data.heads, data.heads.group
    rs = torch.tensor(seqs, device="cuda")
    sc = torch.full((len(seqs), path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, len(seqs), L), dtype=torch.uint8, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, data.q[rs].contiguous(), data.w_q,
                       data.row_seq[rs].contiguous(), data.row_pos[rs].contiguous(), sc, None, None, ws, path.status)
    torch.cuda.synchronize()
    sc = sc.cpu().numpy()
    idx, cnt = path.sel_idx[rs].cpu().numpy(), path.sel_cnt[rs].cpu().numpy()
    out = path.out[rs].float().cpu().numpy()
    qh, w_q, w_k = _np16(data.q[rs]), _np16(data.w_q), _np16(data.w_k)
    for k, b in enumerate(seqs):
        for i, h in enumerate(heads.ret_q_heads):
            c = int(cnt[k, i])
            got = set(idx[k, i, :c].tolist())
            assert len(got) == c
            mand, forb = orc.classify_against_band(sc[k, i], data.top_p)
            assert mand <= got and not (forb & got), f"seq {b} head {i}"
            assert orc.set_mass(sc[k, i], got) >= data.top_p
            kk, vv = data.logical_kv(b, h // g)
            want, _ = orc.attention_over_set(qh[k, h], kk, vv, sorted(got), data.sm_scale)
            assert np.abs(out[k, h] - want).max() <= 2e-2, f"seq {b} head {h}"
            if e2e and i % 4 == 0:
                j = heads.q_head_to_index_head[i]
                kt_o = orc.index_project(data.logical_kv(b, heads.index_head_kv[j])[0], w_k[j])
                ref = orc.retrieval_row(qh[k, h], qh[k, h], w_q[i], kt_o, kk, vv, L - 1, data.top_p, data.score_scale,
                                        data.sm_scale)
                so = ref["scores"]
                qf, kf = orc.bf16_to_f64(ref["qt"]), orc.bf16_to_f64(kt_o)
                tol = 1e-3 * np.abs(so) + 2.0 ** -7 * data.score_scale * (np.abs(kf) @ np.abs(qf))
                _e2e_set_check(so, sc[k, i], got, data.top_p, tol, f"e2e seq {b} head {i}")
                if got == set(ref["ids"].tolist()):
                    assert np.abs(out[k, h] - ref["out"]).max() <= 2e-2, f"e2e output seq {b} head {h}"
        kh = heads.local_kv_heads[0]
        kk, vv = data.logical_kv(b, kh)
        for jj in range(g):
            want, _ = orc.local_row(qh[k, kh * g + jj], kk, vv, L - 1, heads.n_sink, heads.window, data.sm_scale)
            assert np.abs(out[k, kh * g + jj] - want).max() <= 2e-2


def _decode_variant_point(L, B, frac, window, seqs, **variant):
    """The selectable variants at full size: lists of sampled sequences equal the oracle's sets on the GPU's scores,
    attention over them matches the oracle."""
    from paper_2605_16928_b200 import pipeline, synth_device
    data = synth_device.decode_device(L, B, 0.9, frac, window, name="c5_decode_sweep")
    path = pipeline.DecodePath(data, sel_stride=int(min(L, max(16384, 4 * frac * L))), **variant)
    path.build_index_cache()
    k_new = torch.stack([data.k_pre_rows(b, L - 1, L)[0] for b in range(B)]).contiguous()
    path.step(data.q, k_new)
    torch.cuda.synchronize()
    assert path.status_code() == rb.RTP_OK
    heads, g = data.heads, data.heads.group
    rs = torch.tensor(seqs, device="cuda")
    sc = torch.full((len(seqs), path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, len(seqs), L), dtype=torch.uint8, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, data.q[rs].contiguous(), data.w_q,
                       data.row_seq[rs].contiguous(), data.row_pos[rs].contiguous(), sc, None, None, ws, path.status)
    torch.cuda.synchronize()
    sc = sc.cpu().numpy()
    idx, cnt = path.sel_idx[rs].cpu().numpy(), path.sel_cnt[rs].cpu().numpy()
    out = path.out[rs].float().cpu().numpy()
    qh = _np16(data.q[rs])
    top_k, fs, fr = variant.get("top_k", 0), variant.get("force_sink", 0), variant.get("force_recent", 0)
    for k, b in enumerate(seqs):
        for i, h in enumerate(heads.ret_q_heads):
            c = int(cnt[k, i])
            lst = idx[k, i, :c]
            if top_k:
                regular = orc.topk_select(sc[k, i], top_k)[0]
            else:
                thr, tie = float(path.sel_thr[b, i]), int(path.sel_tie[b, i])
                regular = np.nonzero((sc[k, i] > thr) | ((sc[k, i] == thr) & (np.arange(L) <= tie)))[0]
                mand, forb = orc.classify_against_band(sc[k, i], data.top_p)
                assert mand <= set(regular.tolist()) and not (forb & set(regular.tolist()))
            want = orc.with_forced(regular, L - 1, fs, fr)
            assert np.array_equal(np.sort(lst), want), f"seq {b} head {i}"
            kk, vv = data.logical_kv(b, h // g)
            ref, _ = orc.attention_over_set(qh[k, h], kk, vv, want, data.sm_scale)
            assert np.abs(out[k, h] - ref).max() <= 2e-2, f"seq {b} head {h}"


def test_decode_512k_batch4_fixed_budget_4096():
    _decode_variant_point(524288, 4, 0.05, 4096, [1, 2], top_k=4096)


def test_decode_128k_forced_positions():
    _decode_variant_point(131072, 2, 0.05, 4096, [0, 1], force_sink=4, force_recent=256)
    _decode_variant_point(131072, 2, 0.05, 4096, [1], top_k=4096, force_sink=4, force_recent=256)


def test_decode_512k_batch4_8bit_index_keys():
    """The 8-bit index-key cache at full size: sets against the oracle's Top-P on the scores of that cache."""
    _decode_point(524288, 4, 0.9, 0.05, 4096, [0, 2], e2e=False, ikey_e4m3=True)


@pytest.mark.parametrize("L,B,seqs", [(524288, 4, [0, 3]), (1048576, 2, [1])])
def test_decode_block_selection_full_size(L, B, seqs):
    """Block-wise decode at full size (one million keys = 16384 blocks is the most a row may have): page lists of sampled
    sequences against the oracle's block rule on the GPU's scores, attention over the listed pages against the oracle."""
    from paper_2605_16928_b200 import pipeline, synth_device
    data = synth_device.decode_device(L, B, 0.9, 0.05, 4096, name="c5_decode_sweep")
    path = pipeline.DecodePath(data, sel_stride=4096)
    path.build_index_cache()
    k_new = torch.stack([data.k_pre_rows(b, L - 1, L)[0] for b in range(B)]).contiguous()
    path.step_blocks(data.q, k_new)
    torch.cuda.synchronize()
    assert path.status_code() == rb.RTP_OK
    heads, g = data.heads, data.heads.group
    rs = torch.tensor(seqs, device="cuda")
    sc = torch.full((len(seqs), path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, len(seqs), L), dtype=torch.uint8, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, data.q[rs].contiguous(), data.w_q,
                       data.row_seq[rs].contiguous(), data.row_pos[rs].contiguous(), sc, None, None, ws, path.status)
    torch.cuda.synchronize()
    sc = sc.cpu().numpy()
    idx, cnt = path.blk_idx[rs].cpu().numpy(), path.blk_cnt[rs].cpu().numpy()
    out = path.out[rs].float().cpu().numpy()
    qh = _np16(data.q[rs])
    n_b = L // 64
    for k, b in enumerate(seqs):
        for i, h in enumerate(heads.ret_q_heads):
            c = int(cnt[k, i])
            got = set(idx[k, i, :c].tolist())
            assert len(got) == c and 1 <= c <= n_b
            mand, forb = orc.classify_blocks_against_band(sc[k, i], data.top_p)
            assert mand <= got and not (forb & got), f"seq {b} head {i}"
            if i % 4 == 0:
                kk, vv = data.logical_kv(b, h // g)
                want, _ = orc.attention_over_set(qh[k, h], kk, vv, orc.block_token_set(sorted(got), L - 1), data.sm_scale)
                assert np.abs(out[k, h] - want).max() <= 2e-2, f"seq {b} head {h}"


def test_decode_32k_batch8_sampled_rows():
    _decode_point(32768, 8, 0.95, 0.1, 2048, [0, 3, 4, 7], peaked_half=True, name="c2_decode_batched_gqa")


def test_decode_512k_batch4_sampled_rows():
    _decode_point(524288, 4, 0.9, 0.05, 4096, [0, 3])


def test_decode_1m_batch16_sampled_rows():
    _decode_point(1048576, 16, 0.9, 0.01, 4096, [1, 14], e2e=False)


def test_prefill_128k_blocks_sampled_rows():
    """Block-wise top-p (Section 3.4) at the benchmark's size: the last chunk and one from the middle."""
    from paper_2605_16928_b200 import pipeline, synth_device
    L, chunk = 131072, 8192
    data = synth_device.config_3_device(L=L)
    path = pipeline.PrefillPath(data, chunk)
    for s in range(0, L, 131072):
        path.index_keys_range(0, s, min(L, s + 131072))
    heads, g = data.heads, data.heads.group
    rng = np.random.default_rng(11)
    out = torch.zeros((chunk, 32, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((chunk, 32), dtype=torch.float32, device="cuda")
    kv = {}
    for s0 in (6 * chunk, L - chunk):
        path.run_chunk_blocks(s0, chunk, data.q[s0:s0 + chunk], data.k_pre_rows(0, s0, s0 + chunk), out, lse)
        torch.cuda.synchronize()
        assert path.status_code() == rb.RTP_OK
        rows = sorted({s0, s0 + chunk - 1, *map(int, rng.integers(s0, s0 + chunk, 6))})
        sc, _, qh = _gpu_scores(path, data, rows, L)
        r_t = torch.tensor([m - s0 for m in rows], device="cuda")
        mask = path.blk_mask[r_t].cpu().numpy()
        cnt, mass = path.sel_cnt[r_t].cpu().numpy(), path.sel_mass[r_t].cpu().numpy()
        thr, tie = path.sel_thr[r_t].cpu().numpy(), path.sel_tie[r_t].cpu().numpy()
        o_h, l_h = out[r_t].float().cpu().numpy(), lse[r_t].cpu().numpy()
        for k, m in enumerate(rows):
            n_b = m // 64 + 1
            for i, h in enumerate(heads.ret_q_heads):
                s = sc[k, i, : m + 1]
                w = mask[k, i].view(np.uint32)
                got = {b for b in range(n_b) if (int(w[b >> 5]) >> (b & 31)) & 1}
                assert len(got) == int(cnt[k, i])
                mb, lb = orc.block_lse(s)
                assert got == {b for b in range(n_b) if mb[b] > thr[k, i] or (mb[b] == thr[k, i] and b <= tie[k, i])}
                mand, forb = orc.classify_blocks_against_band(s, data.top_p)
                assert mand <= got and not (forb & got), f"row {m} head {i}"
                wgt = lb * np.exp(mb.astype(np.float64) - float(mb.max()))
                tm = float(wgt[sorted(got)].sum() / wgt.sum())
                assert tm >= data.top_p and abs(tm - mass[k, i]) <= 1e-4
                kh = h // g
                if kh not in kv:
                    kv[kh] = data.logical_kv(0, kh)
                want, wlse = orc.attention_over_set(qh[k, h], kv[kh][0], kv[kh][1], orc.block_token_set(sorted(got), m),
                                                    data.sm_scale)
                assert np.abs(o_h[k, h] - want).max() <= 2e-2, f"row {m} head {h}"
                assert abs(l_h[k, h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
