"""GPU parity of the 8-bit (E4M3) index-key cache against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _harness():
    from tests import gpu_harness as gh
    return gh


def _run(wl, rows=None, **kw):
    gh = _harness()
    dw = gh.DeviceWorkload(wl, ikey_e4m3=True, **kw)
    assert dw.cache.ikey_format == rb.RTP_IKEY_E4M3
    dw.index_all_keys()
    gh.check_index_keys(dw)                       # codes against the oracle's encoder
    qt = gh.check_queries(dw)
    sc = gh.check_scores(dw, qt, rows=rows)       # Eq. 4 on the decoded keys
    sel = dw.select()
    stats = gh.check_selection(dw, sc, sel, rows=rows)
    out, lse = dw.sparse_decode()
    gh.check_sparse_attention(dw, sel, out, lse, rows=rows)
    assert dw.status_code() == rb.RTP_OK
    return dw, sc, sel, stats


def _ragged_config2(**kw):
    wl = synth.config_2(L=3000, batch=4, window=512, **kw)
    for b, cut in enumerate([0, 517, 1, 2049]):
        L = 3000 - cut
        wl.k[b], wl.v[b] = wl.k[b][:L], wl.v[b][:L]
        wl.seq_lens[b] = L
        wl.row_pos[b] = L - 1
    return wl


def test_decode_ragged_batch():
    _run(_ragged_config2())


@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 130, 1000])
def test_ragged_lengths(L):
    _run(synth.config_1(L=L, n_needles=min(8, max(1, L // 4))))


def test_group_of_eight_query_heads_per_kv_head():
    _run(synth.config_2(L=2600, batch=2, n_q_heads=16, n_kv_heads=2, ret_kv_heads=(0,), window=300))


def test_fixed_budget_on_8bit_keys():
    gh = _harness()
    wl = _ragged_config2()
    dw = gh.DeviceWorkload(wl, ikey_e4m3=True, top_k=300)
    dw.index_all_keys()
    sc = dw.scores()[0]
    sel = dw.select()
    gh.check_variant_selection(dw, sc, sel, top_k=300)
    assert dw.status_code() == rb.RTP_OK


def test_saturation_and_small_values():
    """Index keys far outside and far inside the 8-bit range: codes saturate at 448 / fall to subnormals and zero, as the
    oracle's encoder says."""
    gh = _harness()
    wl = synth.config_1(L=512, n_needles=4)
    K = synth.from_bf16(wl.k[0])
    K[100:200] *= 4096.0                                       # projections of a few thousand: saturate
    K[300:400] *= 2.0 ** -12                                   # projections near 2^-12: subnormal codes and zeros
    wl.k[0] = synth.to_bf16(K)
    dw = gh.DeviceWorkload(wl, ikey_e4m3=True)
    dw.index_all_keys()
    gh.check_index_keys(dw)
    codes = dw.ikeys_logical(0)[:, 0]
    assert np.any((codes[100:200] & 0x7F) == 0x7E) and np.any((codes[300:400] & 0x78) == 0)
    qt = gh.check_queries(dw)
    gh.check_scores(dw, qt)


def test_8bit_selection_keeps_most_of_the_bf16_mass():
    """Accuracy of the option, not a parity statement: the set chosen on the 8-bit cache, weighed with the scores of the
    bf16 cache, still holds nearly p of the mass on the batched-decode workload."""
    gh = _harness()
    wl = _ragged_config2()
    dw8, sc8, sel8, _ = _run(wl)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    sc = dw.scores()[0]
    from oracle import rtp_oracle as orc
    worst = 1.0
    idx, cnt = sel8["idx"].cpu().numpy(), sel8["cnt"].cpu().numpy()
    for r in range(dw.R):
        m = int(wl.row_pos[r])
        for i in range(dw.n_ret):
            worst = min(worst, orc.set_mass(sc[r, i, : m + 1], idx[r, i, : cnt[r, i]]))
            # scores of the two caches differ by the keys' rounding: 2^-4 relative per element at most
            assert np.abs(sc8[r, i, : m + 1] - sc[r, i, : m + 1]).max() <= 0.07 * np.abs(sc[r, i, : m + 1]).max() + 0.05
    assert worst >= wl.top_p - 0.05, worst


def test_chunk_and_block_forms_need_the_bf16_cache():
    gh = _harness()
    wl = synth.config_3(L=512)
    pr = gh.PrefillRun(gh.DeviceWorkload(wl, ikey_e4m3=True))
    pr.dw.index_all_keys()
    with pytest.raises(rb.RtpError) as e:
        pr.select_chunk(256, 256)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
    sel = dict(idx=None, cnt=torch.zeros((256, pr.n_ret), dtype=torch.int32, device="cuda"),
               thr=torch.zeros((256, pr.n_ret), dtype=torch.float32, device="cuda"),
               tie=torch.zeros((256, pr.n_ret), dtype=torch.int32, device="cuda"))
    with pytest.raises(rb.RtpError) as e:
        pr.sparse_prefill(256, 256, sel, use_lists=False)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
