"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the CUDA path runs
the whole workload, the oracle checks sampled rows one by one."""
import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import binding as rb

pytestmark = pytest.mark.gpu


def _np16(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def test_prefill_128k_sampled_rows():
    from paper_2605_16928_b200 import pipeline, synth_device
    L, chunk = 131072, 8192
    data = synth_device.config_3_device(L=L)
    path = pipeline.PrefillPath(data, chunk)
    heads, g = data.heads, data.heads.group
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
    rows = sorted({0, 1, 63, 64, chunk - 1, chunk, L - 1, L - chunk, *map(int, rng.integers(0, L, 6))})
    # stage-wise parity on the sampled rows: GPU-written index keys and projected queries feed the oracle's
    # scoring; the selection is judged on the GPU's own materialised scores; attention on the GPU's own set
    ik = _np16(path.ikey_pages[data.block_table[0].long()])               # [pages, nih, 64, 16]
    kt = np.transpose(ik, (0, 2, 1, 3)).reshape(-1, heads.n_index_heads, 16)[:L]
    qt = torch.empty((len(rows), path.n_ret, 16), dtype=torch.bfloat16, device="cuda")
    qrows = data.q[torch.tensor(rows, device="cuda")].contiguous()
    rb.rtp_index_queries(path.ctx, path.params, qrows, data.w_q, qt)
    sc = torch.full((len(rows), path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, len(rows), L), dtype=torch.uint8, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, qrows, data.w_q,
                       torch.zeros(len(rows), dtype=torch.int32, device="cuda"),
                       torch.tensor(rows, dtype=torch.int32, device="cuda"), sc, None, None, ws, path.status)
    torch.cuda.synchronize()
    sc = sc.cpu().numpy()
    qt, qh = _np16(qt), _np16(qrows)
    thr_h, tie_h, cnt_h, mass_h = thr.cpu().numpy(), tie.cpu().numpy(), cnt.cpu().numpy(), mass.cpu().numpy()
    out_h, lse_h = out.float().cpu().numpy(), lse.cpu().numpy()
    kv = {}
    fr = []
    for k, m in enumerate(rows):
        for i, h in enumerate(heads.ret_q_heads):
            kh = h // g
            if kh not in kv:
                kv[kh] = data.logical_kv(0, kh)
            s = sc[k, i, : m + 1]
            want_s = orc.index_scores(qt[k, i], kt[: m + 1, heads.q_head_to_index_head[i]], data.score_scale)
            qn = np.linalg.norm(orc.bf16_to_f64(qt[k, i]))
            kn = np.linalg.norm(orc.bf16_to_f64(kt[: m + 1, heads.q_head_to_index_head[i]]), axis=-1)
            assert np.all(np.abs(s - want_s) <= 1e-3 * np.abs(want_s) + 1e-5 * data.score_scale * qn * kn)
            member = (s > thr_h[m, i]) | ((s == thr_h[m, i]) & (np.arange(m + 1) <= tie_h[m, i]))
            got = set(np.nonzero(member)[0].tolist())
            assert len(got) == int(cnt_h[m, i]), f"row {m} head {i}"
            mand, forb = orc.classify_against_band(s, data.top_p)
            assert mand <= got and not (forb & got), f"row {m} head {i}"
            tm = orc.set_mass(s, got)
            assert tm >= data.top_p or len(got) == m + 1
            assert abs(tm - mass_h[m, i]) <= 1e-4
            want, wlse = orc.attention_over_set(qh[k, h], kv[kh][0], kv[kh][1], sorted(got), data.sm_scale)
            assert np.abs(out_h[m, h] - want).max() <= 2e-2, f"sparse row {m} head {h}"
            fr.append(len(got) / (m + 1))
        for kh in heads.local_kv_heads[:2]:
            if kh not in kv:
                kv[kh] = data.logical_kv(0, kh)
            for j in range(g):
                h = kh * g + j
                want, wlse = orc.local_row(qh[k, h], kv[kh][0], kv[kh][1], m, heads.n_sink, heads.window, data.sm_scale)
                assert np.abs(out_h[m, h] - want).max() <= 2e-2, f"local row {m} head {h}"
                assert abs(lse_h[m, h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
    assert 0.002 <= float(np.mean(fr)) <= 0.6


def test_decode_32k_batch8_sampled_rows():
    from paper_2605_16928_b200 import pipeline, synth_device
    L, B = 32768, 8
    data = synth_device.decode_device(L, B, 0.95, 0.1, 2048, peaked_half=True, name="c2_decode_batched_gqa")
    path = pipeline.DecodePath(data, sel_stride=16384)
    path.build_index_cache()
    k_new = torch.stack([data.k_pre_rows(b, L - 1, L)[0] for b in range(B)]).contiguous()
    path.step(data.q, k_new)
    torch.cuda.synchronize()
    assert path.status_code() == rb.RTP_OK
    heads, g = data.heads, data.heads.group
    sc = torch.full((B, path.n_ret, L), float("nan"), dtype=torch.float32, device="cuda")
    rb.rtp_index_score(path.ctx, path.params, path.cache, data.q, data.w_q, data.row_seq, data.row_pos, sc, None, None,
                       path.workspace, path.status)
    sc = sc.cpu().numpy()
    idx, cnt = path.sel_idx.cpu().numpy(), path.sel_cnt.cpu().numpy()
    out = path.out.float().cpu().numpy()
    qh = _np16(data.q)
    for b in [0, 3, 4, 7]:
        for i, h in enumerate(heads.ret_q_heads):
            c = int(cnt[b, i])
            got = set(idx[b, i, :c].tolist())
            assert len(got) == c
            mand, forb = orc.classify_against_band(sc[b, i], data.top_p)
            assert mand <= got and not (forb & got)
            assert orc.set_mass(sc[b, i], got) >= data.top_p
            k, v = data.logical_kv(b, h // g)
            want, _ = orc.attention_over_set(qh[b, h], k, v, sorted(got), data.sm_scale)
            assert np.abs(out[b, h] - want).max() <= 2e-2
        kh = heads.local_kv_heads[0]
        k, v = data.logical_kv(b, kh)
        for j in range(g):
            want, _ = orc.local_row(qh[b, kh * g + j], k, v, L - 1, heads.n_sink, heads.window, data.sm_scale)
            assert np.abs(out[b, kh * g + j] - want).max() <= 2e-2
