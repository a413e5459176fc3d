"""Pins for the oracle's attention, token sets and indexer against library routines."""
import os

import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc
from paper_2605_16928_b200 import synth


def _bf16(rng, shape, scale=1.0):
    return synth.to_bf16((rng.standard_normal(shape) * scale).astype(np.float32))


def _f32(u):
    return torch.from_numpy(synth.from_bf16(u).copy())


def test_bf16_helpers_match_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * 10).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.f32_to_bf16(x), want)
    assert np.array_equal(synth.to_bf16(x), want)
    back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.bf16_to_f64(want), back)


def test_dense_rows_match_sdpa():
    rng = np.random.default_rng(1)
    L = 200
    q, k, v = _bf16(rng, (L, 128)), _bf16(rng, (L, 128)), _bf16(rng, (L, 128))
    ref = torch.nn.functional.scaled_dot_product_attention(
        _f32(q)[None, None].double(), _f32(k)[None, None].double(), _f32(v)[None, None].double(),
        is_causal=True)[0, 0].numpy()
    for m in [0, 1, 63, 64, 65, 199]:
        out, lse = orc.dense_row(q[m], k, v, m, 1.0 / np.sqrt(128))
        assert np.max(np.abs(out - ref[m])) < 1e-9
        logits = (synth.from_bf16(k[: m + 1]).astype(np.float64) @ synth.from_bf16(q[m]).astype(np.float64)) / np.sqrt(128)
        assert lse == pytest.approx(float(torch.logsumexp(torch.from_numpy(logits), 0)), rel=1e-12)


def test_local_rows_match_masked_sdpa():
    rng = np.random.default_rng(2)
    L, n_sink, W = 300, 4, 37
    q, k, v = _bf16(rng, (L, 128)), _bf16(rng, (L, 128)), _bf16(rng, (L, 128))
    i = torch.arange(L)[:, None]
    j = torch.arange(L)[None, :]
    mask = (j <= i) & ((j < n_sink) | (j > i - W))
    ref = torch.nn.functional.scaled_dot_product_attention(
        _f32(q)[None, None].double(), _f32(k)[None, None].double(), _f32(v)[None, None].double(),
        attn_mask=mask[None, None])[0, 0].numpy()
    for m in [0, 3, 4, 36, 37, 40, 41, 299]:
        out, _ = orc.local_row(q[m], k, v, m, n_sink, W, 1.0 / np.sqrt(128))
        assert np.max(np.abs(out - ref[m])) < 1e-9
        assert len(orc.local_set(m, n_sink, W)) == min(m + 1, len(set(range(min(n_sink, m + 1))) | set(range(max(0, m - W + 1), m + 1))))


def test_window_covering_context_equals_dense_and_degenerate_window():
    rng = np.random.default_rng(3)
    L = 150
    q, k, v = _bf16(rng, (L, 128)), _bf16(rng, (L, 128)), _bf16(rng, (L, 128))
    for m in [0, 10, 149]:
        a, la = orc.local_row(q[m], k, v, m, 4, 100000, 0.088)
        b, lb = orc.dense_row(q[m], k, v, m, 0.088)
        assert np.array_equal(a, b) and la == lb
        own, _ = orc.local_row(q[m], k, v, m, 0, 1, 0.088)
        assert np.array_equal(own, orc.bf16_to_f64(v[m]))
    assert orc.local_set(20, 4, 8).tolist() == [0, 1, 2, 3, 13, 14, 15, 16, 17, 18, 19, 20]
    assert orc.local_set(5, 4, 8).tolist() == [0, 1, 2, 3, 4, 5]


def test_sparse_attention_set_properties():
    rng = np.random.default_rng(4)
    L = 500
    q, k, v = _bf16(rng, (128,)), _bf16(rng, (L, 128)), _bf16(rng, (L, 128))
    ids = np.sort(rng.choice(L, 60, replace=False))
    a, la = orc.attention_over_set(q, k, v, ids, 0.088)
    b, lb = orc.attention_over_set(q, k, v, rng.permutation(ids), 0.088)
    assert np.max(np.abs(a - b)) < 1e-12 and la == pytest.approx(lb, rel=1e-12)
    one, _ = orc.attention_over_set(q, k, v, [123], 0.088)
    assert np.array_equal(one, orc.bf16_to_f64(v[123]))
    # log-sum-exp merge of two halves equals the unsplit result (split-KV identity)
    o1, l1 = orc.attention_over_set(q, k, v, ids[:25], 0.088)
    o2, l2 = orc.attention_over_set(q, k, v, ids[25:], 0.088)
    lm = np.logaddexp(l1, l2)
    merged = o1 * np.exp(l1 - lm) + o2 * np.exp(l2 - lm)
    assert np.max(np.abs(merged - a)) < 1e-12 and lm == pytest.approx(la, rel=1e-12)


def test_top_p_one_equals_dense_causal():
    rng = np.random.default_rng(5)
    L = 120
    wq, wk = _bf16(rng, (128, 16), 0.09), _bf16(rng, (128, 16), 0.09)
    q, k, v = _bf16(rng, (L, 128)), _bf16(rng, (L, 128)), _bf16(rng, (L, 128))
    kt = orc.index_project(k, wk)
    for m in [0, 17, 119]:
        r = orc.retrieval_row(q[m], q[m], wq, kt, k, v, m, 1.0, 1.0, 0.088)
        d, ld = orc.dense_row(q[m], k, v, m, 0.088)
        assert r["count"] == m + 1 and np.array_equal(r["out"], d) and r["lse"] == ld


def test_indexer_is_the_matrix_product():
    rng = np.random.default_rng(6)
    n, R = 257, 9
    wq, wk = _bf16(rng, (128, 16), 0.09), _bf16(rng, (128, 16), 0.09)
    qp, kp = _bf16(rng, (R, 128)), _bf16(rng, (n, 128))
    kt = orc.index_project(kp, wk)
    qt = orc.index_project(qp, wq)
    # projections: torch float64 GEMM, rounded the same way
    kt_ref = (_f32(kp).double() @ _f32(wk).double()).float().to(torch.bfloat16)
    qt_ref = (_f32(qp).double() @ _f32(wq).double()).float().to(torch.bfloat16)
    assert np.array_equal(kt, kt_ref.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(qt, qt_ref.view(torch.int16).numpy().view(np.uint16))
    S = (qt_ref.double() @ kt_ref.double().T * 0.37).float().numpy()
    for r in range(R):
        s = orc.index_scores(qt[r], kt, 0.37)
        assert s.dtype == np.float32
        np.testing.assert_allclose(s, S[r], rtol=1e-6, atol=1e-7)
    # a transposed weight or a swapped operand must not pass: shape of the product is asymmetric
    full = (_f32(qp).double() @ _f32(wq).double()) @ (_f32(kp).double() @ _f32(wk).double()).T
    np.testing.assert_allclose(S / 0.37, full.numpy(), rtol=0.05, atol=0.5)


def test_golden_table2_defaults():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "table2_config.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    hm = synth.HeadMap(32, 8, [0, 1])
    assert hm.n_sink == vals["sink_tokens"] and hm.window == vals["sliding_window"]
    assert synth.INDEX_DIM == vals["low_dim"] == orc.INDEX_DIM
    assert synth.PAGE_SIZE == vals["kernel_block"]
    assert synth.config_1(L=256).top_p == vals["top_p"]
