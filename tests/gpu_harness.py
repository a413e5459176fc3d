"""Shared helpers for the GPU parity tests: upload a synthetic workload, run the library
through the C ABI binding, and compare stage by stage against the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

DEV = "cuda:0"


def dev_bf16(u16: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(u16).view(np.int16)).to(DEV).view(torch.bfloat16)


def host_u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


class DeviceWorkload:
    def __init__(self, wl: synth.Workload, sel_stride: int | None = None, ikey_e4m3: bool = False, **param_over):
        self.wl = wl
        self.f8 = ikey_e4m3
        self.ctx = rb.Context()
        self.params = rb.Params.from_workload(wl, **param_over)
        self.pc = synth.build_paged_cache(wl.k, wl.v, wl.seed)
        self.k_pages = dev_bf16(self.pc.k_pages)
        self.v_pages = dev_bf16(self.pc.v_pages)
        nih = max(1, wl.heads.n_index_heads)
        # poison the index-key cache so that unwritten slots are noticed
        if ikey_e4m3:   # (0x7f is the NaN code of the 8-bit format)
            self.ikey_pages = torch.full((self.pc.num_pages, nih, 64, 16), 0x7F, dtype=torch.uint8, device=DEV)
        else:
            self.ikey_pages = torch.full((self.pc.num_pages, nih, 64, 16), float("nan"), dtype=torch.bfloat16, device=DEV)
        self.block_table = dev_i32(self.pc.block_table)
        self.seq_lens = dev_i32(self.pc.seq_lens)
        self.cache = rb.make_cache(self.k_pages, self.v_pages, self.ikey_pages, self.block_table, self.seq_lens)
        self.w_q = dev_bf16(wl.w_q)
        self.w_k = dev_bf16(wl.w_k)
        self.q = dev_bf16(wl.q)
        self.row_seq = dev_i32(wl.row_seq)
        self.row_pos = dev_i32(wl.row_pos)
        self.R = int(wl.row_seq.shape[0])
        self.max_len = int(max(int(x) for x in wl.seq_lens))
        self.n_ret = len(wl.heads.ret_q_heads)
        ws_bytes = max(1 << 20, rb.rtp_workspace_bytes(self.params, max(1, self.R), max(1, self.max_len)))
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)
        self.sel_stride = sel_stride if sel_stride is not None else self.max_len
        self.ikey_host = None

    # ---- S0
    def index_all_keys(self, chunk: int = 1 << 16):
        wl = self.wl
        for b in range(wl.batch):
            L = int(wl.seq_lens[b])
            for lo in range(0, L, chunk):
                hi = min(L, lo + chunk)
                kp = dev_bf16(synth.k_pre_for_index_heads(wl, b, lo, hi))
                tok_seq = torch.full((hi - lo,), b, dtype=torch.int32, device=DEV)
                tok_pos = torch.arange(lo, hi, dtype=torch.int32, device=DEV)
                rb.rtp_index_keys(self.ctx, self.params, self.cache, kp, self.w_k, tok_seq, tok_pos)
        torch.cuda.synchronize()
        self.ikey_host = self.ikey_pages.cpu().numpy() if self.f8 else host_u16(self.ikey_pages)

    def ikeys_logical(self, seq: int) -> np.ndarray:
        return synth.gather_index_keys(self.ikey_host, self.pc.block_table, seq, int(self.wl.seq_lens[seq]))

    # ---- S1
    def project_queries(self) -> np.ndarray:
        qt = torch.empty((self.R, self.n_ret, 16), dtype=torch.bfloat16, device=DEV)
        rb.rtp_index_queries(self.ctx, self.params, self.q, self.w_q, qt)
        torch.cuda.synchronize()
        return host_u16(qt)

    # ---- S2/S3
    def scores(self):
        sc = torch.full((self.R, self.n_ret, self.max_len), float("nan"), dtype=torch.float32, device=DEV)
        mx = torch.empty((self.R, self.n_ret), dtype=torch.float32, device=DEV)
        sm = torch.empty((self.R, self.n_ret), dtype=torch.float32, device=DEV)
        rb.rtp_index_score(self.ctx, self.params, self.cache, self.q, self.w_q, self.row_seq, self.row_pos, sc, mx,
                           sm, self.workspace, self.status)
        torch.cuda.synchronize()
        return sc.cpu().numpy(), mx.cpu().numpy(), sm.cpu().numpy()

    # ---- S4
    def select(self, with_lists: bool = True, chunk: tuple | None = None, general_path: bool = False):
        """general_path: force the multi-kernel decode selection where the one-CTA path for short contexts would run."""
        rb.rtp_debug_select_path(self.ctx, 1 if general_path else 0)
        R, n_ret = self.R, self.n_ret
        idx = torch.full((R, n_ret, self.sel_stride), -1, dtype=torch.int32, device=DEV) if with_lists else None
        cnt = torch.full((R, n_ret), -7, dtype=torch.int32, device=DEV)
        mass = torch.zeros((R, n_ret), dtype=torch.float32, device=DEV)
        thr = torch.zeros((R, n_ret), dtype=torch.float32, device=DEV)
        tie = torch.zeros((R, n_ret), dtype=torch.int32, device=DEV)
        if chunk is None:
            rb.rtp_topp_select(self.ctx, self.params, self.cache, self.q, self.w_q, self.row_seq, self.row_pos, 0, 0,
                               R, idx, cnt, mass, thr, tie, self.status, self.workspace)
        else:
            seq_id, q_start = chunk
            rb.rtp_topp_select(self.ctx, self.params, self.cache, self.q, self.w_q, None, None, seq_id, q_start, R,
                               idx, cnt, mass, thr, tie, self.status, self.workspace)
        torch.cuda.synchronize()
        rb.rtp_debug_select_path(self.ctx, 0)
        self.sel = dict(idx=idx, cnt=cnt, mass=mass, thr=thr, tie=tie)
        return self.sel

    # ---- S5
    def sparse_decode(self):
        out = torch.zeros((self.R, self.wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((self.R, self.wl.heads.n_q_heads), dtype=torch.float32, device=DEV)
        rb.rtp_sparse_attn_decode(self.ctx, self.params, self.cache, self.q, self.row_seq, self.row_pos,
                                  self.sel["idx"], self.sel["cnt"], out, lse, self.workspace, self.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def local_decode(self):
        out = torch.zeros((self.R, self.wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((self.R, self.wl.heads.n_q_heads), dtype=torch.float32, device=DEV)
        rb.rtp_local_attn(self.ctx, self.params, self.cache, self.q, self.row_seq, self.row_pos, 0, 0, self.R, out,
                          lse, self.workspace, self.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def dense_decode(self, kv_heads=None):
        out = torch.zeros((self.R, self.wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((self.R, self.wl.heads.n_q_heads), dtype=torch.float32, device=DEV)
        rb.rtp_dense_attn_decode(self.ctx, self.params, self.cache, self.q, self.row_seq, self.row_pos, kv_heads, out,
                                 lse, self.workspace, self.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def status_code(self) -> int:
        return rb.rtp_check_status(self.ctx, self.status)


# ------------------------------------------------------------------ stage checks
def bf16_ulp_diff(a_u16: np.ndarray, b_u16: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two bit patterns (sign-magnitude -> ordered)."""
    def ordered(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, 0x8000 - (u & 0x7FFF) - 1, u + 0x8000)
    return np.abs(ordered(a_u16) - ordered(b_u16))


def check_index_keys(dw: DeviceWorkload):
    wl = dw.wl
    total = equal = 0
    for b in range(wl.batch):
        got = dw.ikeys_logical(b)                                   # [L, nih, 16]
        kp = synth.k_pre_for_index_heads(wl, b)
        for j in range(wl.heads.n_index_heads):
            if dw.f8:
                # E4M3 codes: equal, or one step apart where the fp32 sum lies at a rounding boundary of the 8-bit grid
                want = orc.index_project_e4m3(kp[:, j], wl.w_k[j])
                g8, w8 = got[:, j].astype(np.int32), want.astype(np.int32)
                order = lambda c: np.where(c & 0x80, -(c & 0x7F), c & 0x7F)
                d = np.abs(order(g8) - order(w8))
                assert d.max() <= 1, f"index key off by {d.max()} E4M3 steps"
                assert not np.any((g8 & 0x7F) == 0x7F), "NaN code written"
                total += d.size
                equal += int((d == 0).sum())
                continue
            want = orc.index_project(kp[:, j], wl.w_k[j])
            d = bf16_ulp_diff(got[:, j], want)
            # one bf16 step, except where cancellation leaves a result so small that the fp32
            # accumulation error (a few 2^-24 of the sum of magnitudes) spans several steps
            floor = np.abs(orc.bf16_to_f64(kp[:, j])) @ np.abs(orc.bf16_to_f64(wl.w_k[j])) * 2.0 ** -21
            bad = (d > 1) & (np.abs(orc.bf16_to_f64(got[:, j]) - orc.bf16_to_f64(want)) > floor)
            assert not bad.any(), f"index key off by {d[bad].max()} bf16 steps"
            total += d.size
            equal += int((d == 0).sum())
    assert equal >= 0.999 * total, f"only {equal}/{total} index keys bit-equal"


def check_queries(dw: DeviceWorkload) -> np.ndarray:
    wl = dw.wl
    qt = dw.project_queries()
    for i, h in enumerate(wl.heads.ret_q_heads):
        want = orc.index_project(wl.q[:, h], wl.w_q[i])
        d = bf16_ulp_diff(qt[:, i], want)
        floor = np.abs(orc.bf16_to_f64(wl.q[:, h])) @ np.abs(orc.bf16_to_f64(wl.w_q[i])) * 2.0 ** -21
        bad = (d > 1) & (np.abs(orc.bf16_to_f64(qt[:, i]) - orc.bf16_to_f64(want)) > floor)
        assert not bad.any()
    return qt


def check_scores(dw: DeviceWorkload, qt: np.ndarray, rows=None):
    """GPU scores against the oracle fed with the GPU-written projections."""
    wl = dw.wl
    sc, mx, sm = dw.scores()
    rows = range(dw.R) if rows is None else rows
    for r in rows:
        b, m = int(wl.row_seq[r]), int(wl.row_pos[r])
        kt = dw.ikeys_logical(b)
        for i in range(dw.n_ret):
            j = wl.heads.q_head_to_index_head[i]
            if dw.f8:
                want = orc.index_scores_e4m3(qt[r, i], kt[: m + 1, j], wl.score_scale)
                kn = np.linalg.norm(orc.e4m3_decode(kt[: m + 1, j]), axis=-1)
            else:
                want = orc.index_scores(qt[r, i], kt[: m + 1, j], wl.score_scale)
                kn = np.linalg.norm(orc.bf16_to_f64(kt[: m + 1, j]), axis=-1)
            got = sc[r, i, : m + 1]
            qn = np.linalg.norm(orc.bf16_to_f64(qt[r, i]))
            tol = 1e-3 * np.abs(want) + 1e-5 * wl.score_scale * qn * kn
            assert np.all(np.abs(got - want) <= tol), f"row {r} head {i}: max err {np.abs(got - want).max()}"
            assert np.all(np.isnan(sc[r, i, m + 1:])), "wrote past the causal range"
            M, Z, _ = orc.softmax_mass(got)
            assert mx[r, i] == np.float32(M)
            assert abs(sm[r, i] - Z) <= 2e-5 * Z
    return sc


def check_selection(dw: DeviceWorkload, sc: np.ndarray, sel: dict, rows=None, p: float | None = None):
    """Selected sets against the oracle's top-p run on the GPU's own scores."""
    wl = dw.wl
    p = wl.top_p if p is None else p
    idx = sel["idx"].cpu().numpy() if sel["idx"] is not None else None
    cnt, mass = sel["cnt"].cpu().numpy(), sel["mass"].cpu().numpy()
    thr, tie = sel["thr"].cpu().numpy(), sel["tie"].cpu().numpy()
    rows = range(dw.R) if rows is None else rows
    stats = []
    for r in rows:
        m = int(wl.row_pos[r])
        for i in range(dw.n_ret):
            s = sc[r, i, : m + 1]
            c = int(cnt[r, i])
            assert 1 <= c <= m + 1
            member = (s > thr[r, i]) | ((s == thr[r, i]) & (np.arange(m + 1) <= tie[r, i]))
            assert int(member.sum()) == c, f"row {r} head {i}: threshold rule gives {int(member.sum())}, count {c}"
            got = set(np.nonzero(member)[0].tolist())
            if idx is not None and c <= idx.shape[-1]:
                lst = idx[r, i, :c]
                assert len(set(lst.tolist())) == c, "duplicate ids"
                assert set(lst.tolist()) == got, "list and threshold rule disagree"
                assert np.all(idx[r, i, c:] == -1), "wrote past the count"
            mand, forb = orc.classify_against_band(s, p)
            assert mand <= got, f"row {r} head {i}: {len(mand - got)} mandatory tokens missing"
            assert not (forb & got), f"row {r} head {i}: {len(forb & got)} forbidden tokens selected"
            true_mass = orc.set_mass(s, got)
            assert true_mass >= p or c == m + 1, f"row {r} head {i}: mass {true_mass} < p"
            assert abs(mass[r, i] - true_mass) <= 1e-4
            k_star = orc.topp_select(s, p)[1]
            stats.append((c, k_star, m + 1))
    return stats


def check_variant_selection(dw: DeviceWorkload, sc: np.ndarray, sel: dict, top_k: int = 0, force_sink: int = 0,
                            force_recent: int = 0, rows=None, p: float | None = None):
    """Row lists of the selectable variants (fixed budget, forced positions) against the oracle run on the GPU's own
    scores.  Fixed budget: the regular part is unique, so the lists must be the oracle's sets exactly.  Top-P with forced
    positions: the regular part obeys the band rule of ``check_selection``; the rest is exactly the forced positions
    the regular part left out, and they come last."""
    wl = dw.wl
    p = wl.top_p if p is None else p
    idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
    mass, thr, tie = sel["mass"].cpu().numpy(), sel["thr"].cpu().numpy(), sel["tie"].cpu().numpy()
    rows = range(dw.R) if rows is None else rows
    counts = []
    for r in rows:
        m = int(wl.row_pos[r])
        for i in range(dw.n_ret):
            s = sc[r, i, : m + 1]
            c = int(cnt[r, i])
            assert 1 <= c <= m + 1 and c <= idx.shape[-1]
            lst = idx[r, i, :c]
            assert len(set(lst.tolist())) == c, "duplicate ids"
            assert np.all(idx[r, i, c:] == -1), "wrote past the count"
            member = (s > thr[r, i]) | ((s == thr[r, i]) & (np.arange(m + 1) <= tie[r, i]))
            regular = np.nonzero(member)[0]
            if top_k > 0:
                want_reg, k_taken, want_thr, want_tie = orc.topk_select(s, top_k)
                assert np.array_equal(regular, want_reg), f"row {r} head {i}: regular part differs from the k largest"
                if k_taken <= m:                       # (when every key is taken the threshold outputs are -inf / m)
                    assert thr[r, i] == want_thr and tie[r, i] == want_tie
            else:
                mand, forb = orc.classify_against_band(s, p)
                got = set(regular.tolist())
                assert mand <= got and not (forb & got)
                assert orc.set_mass(s, got) >= p or len(got) == m + 1
            want = orc.with_forced(regular, m, force_sink, force_recent)
            assert c == want.size, f"row {r} head {i}: count {c}, oracle {want.size}"
            assert np.array_equal(np.sort(lst), want)
            assert set(lst[: regular.size].tolist()) == set(regular.tolist()), "forced positions must come last"
            if top_k > 0:
                assert abs(mass[r, i] - c / (m + 1)) <= 1e-6
            else:
                assert abs(mass[r, i] - orc.set_mass(s, want)) <= 1e-4
            counts.append((c, int(regular.size), m + 1))
    return counts


def check_sparse_attention(dw: DeviceWorkload, sel: dict, out: np.ndarray, lse: np.ndarray, rows=None, tol=2e-2):
    wl = dw.wl
    g = wl.heads.group
    idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
    rows = range(dw.R) if rows is None else rows
    worst = 0.0
    for r in rows:
        b = int(wl.row_seq[r])
        for i, h in enumerate(wl.heads.ret_q_heads):
            ids = idx[r, i, : cnt[r, i]]
            want, wl_lse = orc.attention_over_set(wl.q[r, h], wl.k[b][:, h // g], wl.v[b][:, h // g], ids, wl.sm_scale)
            err = np.abs(out[r, h] - want).max()
            worst = max(worst, err)
            assert err <= tol, f"row {r} head {h}: max abs err {err}"
            assert abs(lse[r, h] - wl_lse) <= 1e-3 * max(1.0, abs(wl_lse))
    return worst


def check_range_attention(dw: DeviceWorkload, out, lse, kv_heads, kind: str, rows=None, tol=2e-2):
    wl = dw.wl
    g = wl.heads.group
    rows = range(dw.R) if rows is None else rows
    for r in rows:
        b, m = int(wl.row_seq[r]), int(wl.row_pos[r])
        for kv in kv_heads:
            for j in range(g):
                h = kv * g + j
                if kind == "local" and h in wl.heads.ret_q_heads:
                    continue                      # a retrieval head inside a mixed group: not the local call's
                if kind == "local":
                    want, wlse = orc.local_row(wl.q[r, h], wl.k[b][:, kv], wl.v[b][:, kv], m, wl.heads.n_sink,
                                               wl.heads.window, wl.sm_scale)
                else:
                    want, wlse = orc.dense_row(wl.q[r, h], wl.k[b][:, kv], wl.v[b][:, kv], m, wl.sm_scale)
                err = np.abs(out[r, h] - want).max()
                assert err <= tol, f"{kind} row {r} head {h}: max abs err {err}"
                assert abs(lse[r, h] - wlse) <= 1e-3 * max(1.0, abs(wlse))


# ------------------------------------------------------------------ prefill helpers
class PrefillRun:
    """Chunked prefill of a one-sequence workload whose query rows are positions 0..L-1."""

    def __init__(self, dw: DeviceWorkload):
        self.dw = dw
        wl = dw.wl
        self.L = int(wl.seq_lens[0])
        self.Hq = wl.heads.n_q_heads
        self.n_ret = dw.n_ret

    def select_chunk(self, q_start: int, C: int, with_lists: bool = True, stride: int | None = None):
        dw = self.dw
        stride = stride or (q_start + C)
        idx = torch.full((C, self.n_ret, stride), -1, dtype=torch.int32, device=DEV) if with_lists else None
        cnt = torch.full((C, self.n_ret), -7, dtype=torch.int32, device=DEV)
        mass = torch.zeros((C, self.n_ret), dtype=torch.float32, device=DEV)
        thr = torch.zeros((C, self.n_ret), dtype=torch.float32, device=DEV)
        tie = torch.zeros((C, self.n_ret), dtype=torch.int32, device=DEV)
        q = dw.q[q_start:q_start + C]
        rb.rtp_topp_select(dw.ctx, dw.params, dw.cache, q, dw.w_q, None, None, 0, q_start, C, idx, cnt, mass, thr,
                           tie, dw.status, dw.workspace)
        torch.cuda.synchronize()
        return dict(idx=idx, cnt=cnt, mass=mass, thr=thr, tie=tie)

    def sparse_prefill(self, q_start: int, C: int, sel: dict, use_lists: bool):
        dw = self.dw
        out = torch.zeros((C, self.Hq, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((C, self.Hq), dtype=torch.float32, device=DEV)
        q = dw.q[q_start:q_start + C]
        rb.rtp_sparse_attn_prefill(dw.ctx, dw.params, dw.cache, q, q, dw.w_q, 0, q_start, C,
                                   sel["idx"] if use_lists else None, sel["cnt"], sel["thr"], sel["tie"], out, lse,
                                   dw.workspace, dw.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def local_prefill(self, q_start: int, C: int):
        dw = self.dw
        out = torch.zeros((C, self.Hq, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((C, self.Hq), dtype=torch.float32, device=DEV)
        rb.rtp_local_attn(dw.ctx, dw.params, dw.cache, dw.q[q_start:q_start + C], None, None, 0, q_start, C, out, lse,
                          dw.workspace, dw.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def dense_prefill(self, q_start: int, C: int, kv_heads=None):
        dw = self.dw
        out = torch.zeros((C, self.Hq, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((C, self.Hq), dtype=torch.float32, device=DEV)
        rb.rtp_dense_attn_prefill(dw.ctx, dw.params, dw.cache, dw.q[q_start:q_start + C], 0, q_start, C, kv_heads, out,
                                  lse, dw.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy(), lse.cpu().numpy()

    def scores_for_rows(self, rows):
        """Materialised GPU scores of the given positions (explicit-row entry point)."""
        dw = self.dw
        rows = np.asarray(rows, dtype=np.int32)
        q = dw.q[torch.from_numpy(rows.astype(np.int64)).to(DEV)].contiguous()
        sc = torch.full((len(rows), self.n_ret, self.L), float("nan"), dtype=torch.float32, device=DEV)
        ws = torch.empty(max(1 << 20, rb.rtp_workspace_bytes(dw.params, len(rows), self.L)), dtype=torch.uint8, device=DEV)
        rb.rtp_index_score(dw.ctx, dw.params, dw.cache, q, dw.w_q, dev_i32(np.zeros(len(rows))), dev_i32(rows), sc,
                           None, None, ws, dw.status)
        torch.cuda.synchronize()
        return sc.cpu().numpy()


def check_chunk_selection(pr: PrefillRun, q_start: int, sel: dict, rows, p=None):
    """rows: absolute positions inside the chunk.  Uses the GPU's own scores."""
    wl = pr.dw.wl
    p = wl.top_p if p is None else p
    sc = pr.scores_for_rows(rows)
    idx = sel["idx"].cpu().numpy() if sel["idx"] is not None else None
    cnt, mass = sel["cnt"].cpu().numpy(), sel["mass"].cpu().numpy()
    thr, tie = sel["thr"].cpu().numpy(), sel["tie"].cpu().numpy()
    fracs = []
    for k, m in enumerate(rows):
        r = m - q_start
        for i in range(pr.n_ret):
            s = sc[k, i, : m + 1]
            c = int(cnt[r, i])
            assert 1 <= c <= m + 1, f"row {m} head {i}: count {c}"
            member = (s > thr[r, i]) | ((s == thr[r, i]) & (np.arange(m + 1) <= tie[r, i]))
            assert int(member.sum()) == c, f"row {m} head {i}: rule gives {int(member.sum())}, count {c}"
            got = set(np.nonzero(member)[0].tolist())
            if idx is not None and c <= idx.shape[-1]:
                lst = idx[r, i, :c]
                assert set(lst.tolist()) == got and len(set(lst.tolist())) == c
                assert np.all(idx[r, i, c:] == -1)
            mand, forb = orc.classify_against_band(s, p)
            assert mand <= got, f"row {m} head {i}: {len(mand - got)} mandatory tokens missing"
            assert not (forb & got), f"row {m} head {i}: {len(forb & got)} forbidden tokens selected"
            tm = orc.set_mass(s, got)
            assert tm >= p or c == m + 1
            assert abs(mass[r, i] - tm) <= 1e-4
            fracs.append(c / (m + 1))
    return sc, fracs


def check_prefill_rows(pr: PrefillRun, q_start: int, out, lse, rows, kind: str, kv_heads, sets=None, tol=2e-2):
    """kind: dense | local | sparse (sets[(m, i)] = ids for retrieval head i)."""
    wl = pr.dw.wl
    g = wl.heads.group
    for m in rows:
        r = m - q_start
        if kind == "sparse":
            for i, h in enumerate(wl.heads.ret_q_heads):
                want, wlse = orc.attention_over_set(wl.q[m, h], wl.k[0][:, h // g], wl.v[0][:, h // g], sets[(m, i)],
                                                    wl.sm_scale)
                err = np.abs(out[r, h] - want).max()
                assert err <= tol, f"sparse row {m} head {h}: {err}"
                assert abs(lse[r, h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
            continue
        for kv in kv_heads:
            for j in range(g):
                h = kv * g + j
                if kind == "local" and h in wl.heads.ret_q_heads:
                    continue
                if kind == "local":
                    want, wlse = orc.local_row(wl.q[m, h], wl.k[0][:, kv], wl.v[0][:, kv], m, wl.heads.n_sink,
                                               wl.heads.window, wl.sm_scale)
                else:
                    want, wlse = orc.dense_row(wl.q[m, h], wl.k[0][:, kv], wl.v[0][:, kv], m, wl.sm_scale)
                err = np.abs(out[r, h] - want).max()
                assert err <= tol, f"{kind} row {m} head {h}: {err}"
                assert abs(lse[r, h] - wlse) <= 1e-3 * max(1.0, abs(wlse))
