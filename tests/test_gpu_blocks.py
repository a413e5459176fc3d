"""GPU parity of the block-wise top-p selection (Section 3.4) and of the attention over the selected blocks."""
import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _prep(wl):
    from tests import gpu_harness as gh
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    return gh, dw, gh.PrefillRun(dw)


def select_blocks(dw, q_start, C, L):
    words = ((L + 63) // 64 + 31) // 32
    words = (words + 3) // 4 * 4
    mask = torch.zeros((C, dw.n_ret, words), dtype=torch.int32, device="cuda")
    cnt = torch.full((C, dw.n_ret), -7, dtype=torch.int32, device="cuda")
    mass = torch.zeros((C, dw.n_ret), dtype=torch.float32, device="cuda")
    thr = torch.zeros((C, dw.n_ret), dtype=torch.float32, device="cuda")
    tie = torch.zeros((C, dw.n_ret), dtype=torch.int32, device="cuda")
    ws = torch.empty(rb.rtp_block_workspace_bytes(dw.params, C, q_start + C), dtype=torch.uint8, device="cuda")
    rb.rtp_topp_select_blocks(dw.ctx, dw.params, dw.cache, dw.q[q_start:q_start + C], dw.w_q, 0, q_start, C, mask, cnt, mass,
                              thr, tie, dw.status, ws)
    torch.cuda.synchronize()
    return dict(mask=mask, cnt=cnt, mass=mass, thr=thr, tie=tie)


def blocks_of(mask_row: np.ndarray, n_b: int) -> set:
    w = mask_row.view(np.uint32)
    return {b for b in range(n_b) if (int(w[b >> 5]) >> (b & 31)) & 1}


def check_block_selection(pr, q_start, sel, rows, p):
    """Judged on the GPU's own materialised scores, like the token-level selection."""
    sc = pr.scores_for_rows(rows)
    mask, cnt = sel["mask"].cpu().numpy(), sel["cnt"].cpu().numpy()
    mass, thr, tie = sel["mass"].cpu().numpy(), sel["thr"].cpu().numpy(), sel["tie"].cpu().numpy()
    out = {}
    for k, m in enumerate(rows):
        r = m - q_start
        for i in range(pr.n_ret):
            s = sc[k, i, : m + 1]
            n_b = m // 64 + 1
            got = blocks_of(mask[r, i], n_b)
            assert len(got) == int(cnt[r, i]) and 1 <= len(got) <= n_b, f"row {m} head {i}"
            mb, lb = orc.block_lse(s)
            rule = {b for b in range(n_b) if mb[b] > thr[r, i] or (mb[b] == thr[r, i] and b <= tie[r, i])}
            assert rule == got, f"row {m} head {i}: the (threshold, block) pair does not describe the mask"
            mand, forb = orc.classify_blocks_against_band(s, p)
            assert mand <= got, f"row {m} head {i}: {len(mand - got)} mandatory blocks missing"
            assert not (forb & got), f"row {m} head {i}: {len(forb & got)} forbidden blocks selected"
            w = lb * np.exp(mb.astype(np.float64) - float(mb.max()))
            tm = float(w[sorted(got)].sum() / w.sum())
            assert tm >= p or len(got) == n_b
            assert abs(tm - mass[r, i]) <= 1e-4
            out[(m, i)] = orc.block_token_set(sorted(got), m)
    return out


@pytest.mark.parametrize("make,top_p", [(lambda: synth.config_3(L=3000, window=512), 0.9),
                                        (lambda: synth.config_3(L=3000, window=512, top_p=0.5), 0.5),
                                        (lambda: synth.config_grid_ties(L=3000, amp=2, top_p=0.9), 0.9),
                                        (lambda: synth.config_4(L=4096, n_needles=64), 0.9)])
def test_block_selection_and_attention(make, top_p):
    wl = make()
    gh, dw, pr = _prep(wl)
    L = int(wl.seq_lens[0])
    rng = np.random.default_rng(7)
    bounds = [(0, 1024), (1024, 1024), (2048, L - 2048)]
    fr = []
    for q_start, C in bounds:
        rows = sorted({q_start, q_start + C - 1, q_start + 63, q_start + 64, *map(int, rng.integers(q_start, q_start + C, 5))})
        sel = select_blocks(dw, q_start, C, L)
        sets = check_block_selection(pr, q_start, sel, rows, top_p)
        out = torch.zeros((C, wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((C, wl.heads.n_q_heads), dtype=torch.float32, device="cuda")
        rb.rtp_sparse_attn_prefill_blocks(dw.ctx, dw.params, dw.cache, dw.q[q_start:q_start + C], 0, q_start, C, sel["mask"],
                                          out, lse, dw.status)
        torch.cuda.synchronize()
        gh.check_prefill_rows(pr, q_start, out.float().cpu().numpy(), lse.cpu().numpy(), rows, "sparse", None, sets)
        fr += [len(v) / (m + 1) for (m, i), v in sets.items()]
    assert dw.status_code() == rb.RTP_OK
    assert 0.0 < np.mean(fr) <= 1.0


def test_block_selection_p_one_and_tiny_rows():
    wl = synth.config_3(L=200, window=64, top_p=1.0)
    gh, dw, pr = _prep(wl)
    sel = select_blocks(dw, 0, 200, 200)
    cnt = sel["cnt"].cpu().numpy()
    want = (np.arange(200) // 64 + 1)[:, None]
    assert np.array_equal(cnt, np.broadcast_to(want, cnt.shape))
    assert dw.status_code() == rb.RTP_OK
