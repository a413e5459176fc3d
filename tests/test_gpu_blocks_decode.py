"""GPU parity of the block-wise top-p selection for decode rows (Section 3.4) and of the attention over the selected
pages, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as gh
    return gh


def select_block_rows(dw, stride=None, with_lists=True):
    n_b_max = (dw.max_len + 63) // 64
    stride = stride or n_b_max
    R, n_ret = dw.R, dw.n_ret
    idx = torch.full((R, n_ret, stride), -1, dtype=torch.int32, device="cuda") if with_lists else None
    cnt = torch.full((R, n_ret), -7, dtype=torch.int32, device="cuda")
    mass = torch.zeros((R, n_ret), dtype=torch.float32, device="cuda")
    thr = torch.zeros((R, n_ret), dtype=torch.float32, device="cuda")
    tie = torch.zeros((R, n_ret), dtype=torch.int32, device="cuda")
    ws = torch.empty(max(1 << 16, rb.rtp_block_workspace_bytes(dw.params, max(1, R), max(1, dw.max_len))), dtype=torch.uint8,
                     device="cuda")
    rb.rtp_topp_select_blocks_rows(dw.ctx, dw.params, dw.cache, dw.q, dw.w_q, dw.row_seq, dw.row_pos, idx, cnt, mass, thr,
                                   tie, dw.status, ws)
    torch.cuda.synchronize()
    return dict(idx=idx, cnt=cnt, mass=mass, thr=thr, tie=tie)


def check_block_rows(dw, sc, sel, p, rows=None):
    """Judged on the GPU's own materialised scores, like every other selection."""
    wl = dw.wl
    idx, cnt = sel["idx"].cpu().numpy(), sel["cnt"].cpu().numpy()
    mass, thr, tie = sel["mass"].cpu().numpy(), sel["thr"].cpu().numpy(), sel["tie"].cpu().numpy()
    sets = {}
    for r in (range(dw.R) if rows is None else rows):
        m = int(wl.row_pos[r])
        n_b = m // 64 + 1
        for i in range(dw.n_ret):
            s = sc[r, i, : m + 1]
            c = int(cnt[r, i])
            assert 1 <= c <= n_b, f"row {r} head {i}: count {c}"
            lst = idx[r, i, :c]
            got = set(lst.tolist())
            assert len(got) == c and min(got) >= 0 and max(got) < n_b, "duplicate or out-of-range pages"
            assert np.all(idx[r, i, c:] == -1), "wrote past the count"
            mb, lb = orc.block_lse(s)
            rule = {b for b in range(n_b) if mb[b] > thr[r, i] or (mb[b] == thr[r, i] and b <= tie[r, i])}
            assert rule == got, f"row {r} head {i}: the (threshold, block) pair does not describe the list"
            mand, forb = orc.classify_blocks_against_band(s, p)
            assert mand <= got, f"row {r} head {i}: {len(mand - got)} mandatory blocks missing"
            assert not (forb & got), f"row {r} head {i}: {len(forb & got)} forbidden blocks selected"
            w = lb * np.exp(mb.astype(np.float64) - float(mb.max()))
            tm = float(w[sorted(got)].sum() / w.sum())
            assert tm >= p or c == n_b
            assert abs(tm - mass[r, i]) <= 1e-4
            sets[(r, i)] = orc.block_token_set(sorted(got), m)
    return sets


def attend_blocks(dw, sel, per_head=False):
    """per_head: a workspace too small for the union lists, so that every head gathers its own pages."""
    out = torch.zeros((dw.R, dw.wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((dw.R, dw.wl.heads.n_q_heads), dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda") if per_head else dw.workspace
    rb.rtp_sparse_attn_decode_blocks(dw.ctx, dw.params, dw.cache, dw.q, dw.row_seq, dw.row_pos, sel["idx"], sel["cnt"], out,
                                     lse, ws, dw.status)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), lse.cpu().numpy()


def check_block_attention(dw, sets, out, lse, rows=None, tol=2e-2):
    wl = dw.wl
    g = wl.heads.group
    for r in (range(dw.R) if rows is None else rows):
        b = int(wl.row_seq[r])
        for i, h in enumerate(wl.heads.ret_q_heads):
            want, wl_lse = orc.attention_over_set(wl.q[r, h], wl.k[b][:, h // g], wl.v[b][:, h // g], sets[(r, i)], wl.sm_scale)
            assert np.abs(out[r, h] - want).max() <= tol, f"row {r} head {h}"
            assert abs(lse[r, h] - wl_lse) <= 1e-3 * max(1.0, abs(wl_lse))


def _run(wl, p=None, **kw):
    gh = _harness()
    dw = gh.DeviceWorkload(wl, **kw)
    dw.index_all_keys()
    sc = dw.scores()[0]
    sel = select_block_rows(dw)
    sets = check_block_rows(dw, sc, sel, wl.top_p if p is None else p)
    out, lse = attend_blocks(dw, sel)                       # the group over the union of its heads' pages
    check_block_attention(dw, sets, out, lse)
    local = [h for h in range(wl.heads.n_q_heads) if h not in wl.heads.ret_q_heads]
    assert np.all(out[:, local] == 0), "only retrieval heads are written"
    out, lse = attend_blocks(dw, sel, per_head=True)        # every head over its own pages
    check_block_attention(dw, sets, out, lse)
    assert dw.status_code() == rb.RTP_OK
    return dw, sel, sets


def _ragged_config2(**kw):
    wl = synth.config_2(L=3000, batch=4, window=512, **kw)
    for b, cut in enumerate([0, 517, 1, 2049]):
        L = 3000 - cut
        wl.k[b], wl.v[b] = wl.k[b][:L], wl.v[b][:L]
        wl.seq_lens[b] = L
        wl.row_pos[b] = L - 1
    return wl


def test_ragged_batch_peaked_and_flat_rows():
    dw, sel, sets = _run(_ragged_config2())
    cnt = sel["cnt"].cpu().numpy()
    assert cnt[:2].mean() < cnt[2:].mean()            # peaked rows need fewer blocks than flat ones


@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 130, 1000, 4096])
def test_ragged_lengths(L):
    _run(synth.config_1(L=L, n_needles=min(8, max(1, L // 4))))


def test_group_of_eight_query_heads_per_kv_head():
    _run(synth.config_2(L=2600, batch=2, n_q_heads=16, n_kv_heads=2, ret_kv_heads=(0,), window=300))


def test_mixed_group_block_decode():
    """Two of the four query heads of a KV head are retrieval heads: the union pass computes the group and writes two."""
    _run(synth.config_2(L=3000, batch=2, window=512, ret_per_group=2))


def test_on_8bit_index_keys():
    _run(_ragged_config2(), ikey_e4m3=True)


@pytest.mark.parametrize("p", [0.5, 1.0])
def test_other_thresholds(p):
    dw, sel, sets = _run(_ragged_config2(top_p=p), p=p)
    if p == 1.0:
        n_b = (np.asarray(dw.wl.row_pos) // 64 + 1)[:, None]
        assert np.array_equal(sel["cnt"].cpu().numpy(), np.broadcast_to(n_b, (dw.R, dw.n_ret)))


def test_equal_blocks_take_the_lowest_block_numbers():
    """All index keys equal: every block has the same maximum; full blocks carry equal mass, so the first ceil(p N_b)
    blocks are taken (the row's last, shorter block would come after them anyway)."""
    gh = _harness()
    L = 64 * 47                                                   # (0.9 x 47 is not a whole number of blocks)
    wl = synth.config_1(L=L)
    wl.k[0][:, 0, :] = wl.k[0][0, 0, :]
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    sc = dw.scores()[0]
    sel = select_block_rows(dw)
    c = int(sel["cnt"][0, 0])
    assert c == 43 and sorted(sel["idx"][0, 0, :c].cpu().numpy().tolist()) == list(range(43))
    check_block_rows(dw, sc, sel, wl.top_p)


def test_short_list_reports_capacity_and_bad_pages_are_refused():
    gh = _harness()
    wl = _ragged_config2()
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    sel = select_block_rows(dw, stride=2)
    assert int(sel["cnt"].max()) > 2 and dw.status_code() == rb.RTP_ERR_CAPACITY
    dw.status.zero_()
    sel = select_block_rows(dw)
    bad = sel["idx"].clone()
    bad[1, 0, 0] = 10 ** 6                                        # beyond the row's causal pages
    out, lse = attend_blocks(dw, dict(idx=bad, cnt=sel["cnt"]))
    assert dw.status_code() == rb.RTP_ERR_INVALID


def test_counts_only_and_variants_are_refused():
    gh = _harness()
    wl = _ragged_config2()
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    a = select_block_rows(dw)
    b = select_block_rows(dw, with_lists=False)
    assert torch.equal(a["cnt"], b["cnt"]) and torch.equal(a["thr"], b["thr"])
    dwk = gh.DeviceWorkload(wl, top_k=64)
    dwk.index_all_keys()
    with pytest.raises(rb.RtpError) as e:
        select_block_rows(dwk)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
