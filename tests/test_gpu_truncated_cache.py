"""Local heads on a truncated cache (Sections 1 and 3.2: the full KV cache is kept for retrieval heads only): the same
calls on a cache whose local heads keep only their sink pages and a ring of recent pages must give bit-identical
results to the untruncated cache, in decode and in chunked prefill; the retrieval heads read the smaller main pool."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def _truncated(dw, ring_pages: int, sink_pages: int = 1, seed: int = 5):
    """An empty truncated cache for dw's workload: main pool with the non-local heads on dw's block table, local pool
    behind a shuffled table of sink_pages + ring_pages entries per sequence."""
    wl = dw.wl
    n_loc = len(wl.heads.local_kv_heads)
    n_main = wl.heads.n_kv_heads - n_loc
    B = wl.batch
    slots = sink_pages + ring_pages
    g = torch.Generator(device="cpu").manual_seed(seed)
    perm = torch.randperm(B * slots + 3, generator=g)[: B * slots].to(torch.int32).reshape(B, slots).cuda()
    nan = float("nan")
    k_main = torch.full((dw.pc.num_pages, max(1, n_main), 64, 128), nan, dtype=torch.bfloat16, device="cuda")
    v_main = torch.full_like(k_main, nan)
    k_loc = torch.full((B * slots + 3, n_loc, 64, 128), nan, dtype=torch.bfloat16, device="cuda")
    v_loc = torch.full_like(k_loc, nan)
    cache = rb.make_cache(k_main, v_main, dw.ikey_pages, dw.block_table, dw.seq_lens, k_loc, v_loc, perm, sink_pages)
    keep = (k_main, v_main, k_loc, v_loc, perm)
    return cache, keep


def _append(dw, cache, b, lo, hi):
    from tests import gpu_harness as gh
    k = gh.dev_bf16(dw.wl.k[b][lo:hi])
    v = gh.dev_bf16(dw.wl.v[b][lo:hi])
    tok_seq = torch.full((hi - lo,), b, dtype=torch.int32, device="cuda")
    tok_pos = torch.arange(lo, hi, dtype=torch.int32, device="cuda")
    rb.rtp_kv_append(dw.ctx, dw.params, cache, k, v, tok_seq, tok_pos, dw.status)


def test_decode_on_truncated_cache_is_bit_identical():
    from tests import gpu_harness as gh
    wl = synth.config_5(L=6000, batch=3, top_p=0.9, frac=0.1, window=1024)
    dw = gh.DeviceWorkload(wl, sel_stride=4096)
    dw.index_all_keys()
    dw.select()
    ref_local, ref_lse = dw.local_decode()
    ref_sparse, ref_slse = dw.sparse_decode()
    cache, keep = _truncated(dw, ring_pages=1024 // 64 + 1)
    for b in range(wl.batch):
        for lo in range(0, 6000, 1000):                      # the ring wraps several times (one call never carries more
            _append(dw, cache, b, lo, min(6000, lo + 1000))  # tokens of a sequence than the ring holds)
    H = wl.heads.n_q_heads
    out = torch.zeros((dw.R, H, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((dw.R, H), dtype=torch.float32, device="cuda")
    rb.rtp_local_attn(dw.ctx, dw.params, cache, dw.q, dw.row_seq, dw.row_pos, 0, 0, dw.R, out, lse, dw.workspace, dw.status)
    rb.rtp_sparse_attn_decode(dw.ctx, dw.params, cache, dw.q, dw.row_seq, dw.row_pos, dw.sel["idx"], dw.sel["cnt"], out, lse,
                              dw.workspace, dw.status)
    torch.cuda.synchronize()
    assert dw.status_code() == rb.RTP_OK
    got, got_lse = out.float().cpu().numpy(), lse.cpu().numpy()
    g = wl.heads.group
    loc = [kv * g + j for kv in wl.heads.local_kv_heads for j in range(g)]
    ret = wl.heads.ret_q_heads
    assert np.array_equal(got[:, loc], ref_local[:, loc]) and np.array_equal(got_lse[:, loc], ref_lse[:, loc])
    assert np.array_equal(got[:, ret], ref_sparse[:, ret]) and np.array_equal(got_lse[:, ret], ref_slse[:, ret])
    # what the truncation saves: bytes of K and V held per sequence
    full = 2 * dw.pc.num_pages * wl.heads.n_kv_heads * 64 * 128 * 2
    trunc = 2 * (keep[0].numel() + keep[2].numel()) * 2
    assert trunc < 0.5 * full


def test_chunked_prefill_on_truncated_cache_is_bit_identical():
    from tests import gpu_harness as gh
    wl = synth.config_3(L=3000, window=512)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    pr = gh.PrefillRun(dw)
    chunk = 600
    cache, keep = _truncated(dw, ring_pages=(512 + chunk) // 64 + 2)
    H = wl.heads.n_q_heads
    for q_start in range(0, 3000, chunk):
        C = min(chunk, 3000 - q_start)
        ref, ref_lse = pr.local_prefill(q_start, C)
        _append(dw, cache, 0, q_start, q_start + C)
        out = torch.zeros((C, H, 128), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((C, H), dtype=torch.float32, device="cuda")
        rb.rtp_local_attn(dw.ctx, dw.params, cache, dw.q[q_start:q_start + C], None, None, 0, q_start, C, out, lse,
                          dw.workspace, dw.status)
        sel = pr.select_chunk(q_start, C, with_lists=False)
        ref_s, ref_slse = pr.sparse_prefill(q_start, C, sel, use_lists=False)
        rb.rtp_sparse_attn_prefill(dw.ctx, dw.params, cache, dw.q[q_start:q_start + C], dw.q[q_start:q_start + C], dw.w_q, 0,
                                   q_start, C, None, sel["cnt"], sel["thr"], sel["tie"], out, lse, dw.workspace, dw.status)
        torch.cuda.synchronize()
        got, got_lse = out.float().cpu().numpy(), lse.cpu().numpy()
        g = wl.heads.group
        loc = [kv * g + j for kv in wl.heads.local_kv_heads for j in range(g)]
        ret = wl.heads.ret_q_heads
        assert np.array_equal(got[:, loc], ref[:, loc]) and np.array_equal(got_lse[:, loc], ref_lse[:, loc]), f"chunk at {q_start}"
        assert np.array_equal(got[:, ret], ref_s[:, ret]) and np.array_equal(got_lse[:, ret], ref_slse[:, ret]), f"chunk at {q_start}"
    assert dw.status_code() == rb.RTP_OK


def test_truncated_cache_argument_checks():
    from tests import gpu_harness as gh
    wl = synth.config_3(L=1000, window=512)
    dw = gh.DeviceWorkload(wl)
    cache, keep = _truncated(dw, ring_pages=4)                # 256 tokens: smaller than the window
    out = torch.zeros((8, wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rb.RtpError) as e:
        rb.rtp_local_attn(dw.ctx, dw.params, cache, dw.q[:8], None, None, 0, 0, 8, out, None, dw.workspace, dw.status)
    assert e.value.code == rb.RTP_ERR_CAPACITY
    with pytest.raises(rb.RtpError) as e:                     # a dense call on heads that the main pool does not hold
        rb.rtp_dense_attn_prefill(dw.ctx, dw.params, cache, dw.q[:8], 0, 0, 8, None, out, None, dw.status)
    assert e.value.code == rb.RTP_ERR_UNSUPPORTED
