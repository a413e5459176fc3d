"""The workspace-free sparse decode entry point against the ordinary one.

Some hosts cannot give the library scratch memory at call time (their device heap belongs to a pool
they do not control, or cudaMalloc is off limits where the call is made).  For them
rtp_sparse_attn_decode_static keeps its split partials in a fixed array inside the library.  This test
calls it twice in a row through the C ABI and checks both results against rtp_sparse_attn_decode, then
checks that a call too large for the built-in array is refused with a clear message.  It runs last so
that a failure here cannot hide the other tests' results.
"""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    from tests import gpu_harness as gh
    wl = synth.config_5(L=20000, batch=3, top_p=0.9, frac=0.2)
    dw = gh.DeviceWorkload(wl, sel_stride=8192)
    dw.index_all_keys()
    sel = dw.select()
    assert int(sel["cnt"].max()) > 1000                                  # long lists: the call is split
    ref_out, ref_lse = dw.sparse_decode()
    h = wl.heads.ret_q_heads
    for attempt in range(2):
        out = torch.zeros((dw.R, wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((dw.R, wl.heads.n_q_heads), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]                       # cudaMemGetInfo: device-wide free bytes
        rb.rtp_sparse_attn_decode_static(dw.ctx, dw.params, dw.cache, dw.q, dw.row_seq, dw.row_pos, sel["idx"],
                                         sel["cnt"], out, lse, dw.status)
        torch.cuda.synchronize()
        if attempt == 1:                                                 # (the first call may load the kernel's code)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        got = out.float().cpu().numpy()
        assert np.abs(got[:, h] - ref_out[:, h]).max() <= 2e-2, f"call {attempt}"
        np.testing.assert_allclose(lse.cpu().numpy()[:, h], ref_lse[:, h], rtol=1e-3, atol=1e-3)
        # and against the oracle, like every other attention test
        gh.check_sparse_attention(dw, sel, got, lse.cpu().numpy())
        # a different selection in between, so that the second call really overwrites the first one's partials
        if attempt == 0:
            sel["cnt"] = torch.clamp(sel["cnt"] - 7, min=1)
            dw.sel = sel
            ref_out, ref_lse = dw.sparse_decode()
    assert dw.status_code() == rb.RTP_OK


def test_static_scratch_rejects_oversized_calls():
    from tests import gpu_harness as gh
    wl = synth.config_5(L=4096, batch=2, top_p=0.9, frac=0.2)
    dw = gh.DeviceWorkload(wl)
    R = 70                                                               # 70 rows x 8 heads x 2 splits x 520 B > 512 KiB
    q = dw.q[:1].expand(R, -1, -1).contiguous()
    row_seq = torch.zeros(R, dtype=torch.int32, device="cuda")
    row_pos = torch.full((R,), 4095, dtype=torch.int32, device="cuda")
    idx = torch.zeros((R, dw.n_ret, 1024), dtype=torch.int32, device="cuda")
    cnt = torch.full((R, dw.n_ret), 1024, dtype=torch.int32, device="cuda")
    out = torch.zeros((R, wl.heads.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rb.RtpError) as e:
        rb.rtp_sparse_attn_decode_static(dw.ctx, dw.params, dw.cache, q, row_seq, row_pos, idx, cnt, out, None,
                                         dw.status)
    assert e.value.code == rb.RTP_ERR_CAPACITY and "bytes" in str(e.value)
