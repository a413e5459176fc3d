"""A bounded device-side wait that runs out: the kernel must record RTP_ERR_TIMEOUT in the status word, return,
free its tensor memory, and leave the context usable (no trap, no hang)."""
import numpy as np
import pytest
import torch

from paper_2605_16928_b200 import binding as rb
from paper_2605_16928_b200 import synth

pytestmark = pytest.mark.gpu


def test_withheld_signal_times_out_and_next_call_is_fine():
    from tests import gpu_harness as gh
    wl = synth.config_3(L=300, window=128)
    dw = gh.DeviceWorkload(wl)
    dw.index_all_keys()
    pr = gh.PrefillRun(dw)
    rows = [0, 63, 64, 128, 299]
    out, lse = pr.dense_prefill(0, 300, kv_heads=[0])
    gh.check_prefill_rows(pr, 0, out, lse, rows, "dense", [0])
    assert dw.status_code() == rb.RTP_OK
    # every wait gives up after 3 ms and the key loader never signals its first tile
    rb.rtp_debug_wait_test(dw.ctx, 3_000_000, True)
    try:
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        pr.dense_prefill(0, 300, kv_heads=[0])
        t1.record()
        t1.synchronize()
        assert dw.status_code() == rb.RTP_ERR_TIMEOUT
        assert t0.elapsed_time(t1) < 2000.0          # it gave up: bounded by a few wait limits, not seconds
    finally:
        rb.rtp_debug_wait_test(dw.ctx, 2_000_000_000, False)
    # the context, the caches and the tensor memory are intact: the same call passes parity again
    dw.status.zero_()
    out, lse = pr.dense_prefill(0, 300, kv_heads=[0])
    gh.check_prefill_rows(pr, 0, out, lse, rows, "dense", [0])
    out, lse = pr.local_prefill(0, 300)
    gh.check_prefill_rows(pr, 0, out, lse, rows, "local", wl.heads.local_kv_heads[:1])
    assert dw.status_code() == rb.RTP_OK


def test_wait_test_rejects_bad_arguments():
    ctx = rb.Context()
    with pytest.raises(rb.RtpError):
        rb.rtp_debug_wait_test(ctx, 0, False)
