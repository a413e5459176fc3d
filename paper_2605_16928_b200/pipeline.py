"""Call sequences of the hot path over a ``DeviceData`` workload: buffer allocation and the order of
the C-ABI calls only (no arithmetic happens here).

``PrefillPath.run_chunk`` is one chunk of a chunked prefill (append index keys -> top-p thresholds ->
sparse attention on retrieval heads -> sink+window attention on local heads); ``DecodePath.step`` is
one decode step (append index key -> top-p lists -> sparse attention -> local attention), and both
offer the dense comparator.
"""
from __future__ import annotations

import torch

from . import binding as rb


class _Base:
    def __init__(self, data, max_rows: int, max_len: int, ikey_e4m3: bool = False, **param_over):
        """ikey_e4m3: the index-key cache holds 8-bit floats (16 bytes per token and index head) instead of bf16."""
        self.data = data
        dev = data.q.device
        self.dev = dev
        self.ctx = rb.Context()
        self.params = rb.Params.from_workload(data, **param_over)
        nih = max(1, data.heads.n_index_heads)
        self.ikey_pages = torch.zeros((data.num_pages, nih, 64, 16),
                                      dtype=torch.uint8 if ikey_e4m3 else torch.bfloat16, device=dev)
        self.cache = rb.make_cache(data.k_pages, data.v_pages, self.ikey_pages, data.block_table, data.seq_lens)
        ws = max(1 << 20, rb.rtp_workspace_bytes(self.params, max_rows, max_len))
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.n_ret = len(data.heads.ret_q_heads)
        self.Hq = data.heads.n_q_heads

    def status_code(self) -> int:
        return rb.rtp_check_status(self.ctx, self.status)

    def index_keys_range(self, seq: int, lo: int, hi: int, k_pre=None):
        d = self.data
        k_pre = d.k_pre_rows(seq, lo, hi) if k_pre is None else k_pre
        tok_seq = torch.full((hi - lo,), seq, dtype=torch.int32, device=self.dev)
        tok_pos = torch.arange(lo, hi, dtype=torch.int32, device=self.dev)
        rb.rtp_index_keys(self.ctx, self.params, self.cache, k_pre, d.w_k, tok_seq, tok_pos)


class PrefillPath(_Base):
    """One sequence, rows = positions.  Buffers are sized for one chunk."""

    def __init__(self, data, chunk: int):
        L = int(data.seq_lens[0])
        super().__init__(data, chunk, L)
        self.L, self.chunk = L, chunk
        self.sel_cnt = torch.empty((chunk, self.n_ret), dtype=torch.int32, device=self.dev)
        self.sel_mass = torch.empty((chunk, self.n_ret), dtype=torch.float32, device=self.dev)
        self.sel_thr = torch.empty((chunk, self.n_ret), dtype=torch.float32, device=self.dev)
        self.sel_tie = torch.empty((chunk, self.n_ret), dtype=torch.int32, device=self.dev)
        self.tok_seq = torch.zeros(chunk, dtype=torch.int32, device=self.dev)
        self.pos_all = torch.arange(L, dtype=torch.int32, device=self.dev)
        self.launches_per_chunk = 6   # index_keys, 2 x query projection, select, sparse attention, local attention
        self.blk_mask = None          # block-wise path (Section 3.4): allocated on first use

    def chunks(self):
        return [(s, min(self.chunk, self.L - s)) for s in range(0, self.L, self.chunk)]

    def run_chunk(self, q_start: int, C: int, q, k_pre, out, lse=None):
        """q: bf16 [C, Hq, 128] (also used as q_pre: no RoPE in the synthetic workloads);
        k_pre: bf16 [C, n_index_heads, 128]; out: bf16 [C, Hq, 128]."""
        d, p = self.data, self.params
        rb.rtp_index_keys(self.ctx, p, self.cache, k_pre, d.w_k, self.tok_seq[:C], self.pos_all[q_start:q_start + C])
        rb.rtp_topp_select(self.ctx, p, self.cache, q, d.w_q, None, None, 0, q_start, C, None, self.sel_cnt,
                           self.sel_mass, self.sel_thr, self.sel_tie, self.status, self.workspace)
        rb.rtp_sparse_attn_prefill(self.ctx, p, self.cache, q, q, d.w_q, 0, q_start, C, None, self.sel_cnt,
                                   self.sel_thr, self.sel_tie, out, lse, self.workspace, self.status)
        rb.rtp_local_attn(self.ctx, p, self.cache, q, None, None, 0, q_start, C, out, lse, self.workspace, self.status)

    def run_chunk_blocks(self, q_start: int, C: int, q, k_pre, out, lse=None):
        """The same chunk with the block-wise selection of Section 3.4 on the retrieval heads: append index keys ->
        one bit per (row, head, page) -> attention over the selected pages -> sink + window attention on local heads."""
        d, p = self.data, self.params
        if self.blk_mask is None:
            words = (((self.L + 63) // 64 + 31) // 32 + 3) // 4 * 4
            self.blk_mask = torch.zeros((self.chunk, self.n_ret, words), dtype=torch.int32, device=self.dev)
            self.blk_ws = torch.empty(rb.rtp_block_workspace_bytes(p, self.chunk, self.L), dtype=torch.uint8, device=self.dev)
        rb.rtp_index_keys(self.ctx, p, self.cache, k_pre, d.w_k, self.tok_seq[:C], self.pos_all[q_start:q_start + C])
        rb.rtp_topp_select_blocks(self.ctx, p, self.cache, q, d.w_q, 0, q_start, C, self.blk_mask[:C], self.sel_cnt[:C],
                                  self.sel_mass[:C], self.sel_thr[:C], self.sel_tie[:C], self.status, self.blk_ws)
        rb.rtp_sparse_attn_prefill_blocks(self.ctx, p, self.cache, q, 0, q_start, C, self.blk_mask[:C], out, lse, self.status)
        rb.rtp_local_attn(self.ctx, p, self.cache, q, None, None, 0, q_start, C, out, lse, self.workspace, self.status)

    def run_chunk_dense(self, q_start: int, C: int, q, out, lse=None):
        rb.rtp_dense_attn_prefill(self.ctx, self.params, self.cache, q, 0, q_start, C, None, out, lse, self.status)


class DecodePath(_Base):
    """One decode step for a batch: row b is the newest token of sequence b."""

    def __init__(self, data, sel_stride: int, **param_over):
        """param_over: rtp_params fields that replace the workload's (top_k, force_sink, force_recent, top_p ...)."""
        B = int(data.seq_lens.shape[0])
        L = int(data.seq_lens.max())
        super().__init__(data, B, L, **param_over)
        self.B, self.L = B, L
        self.sel_idx = torch.empty((B, self.n_ret, sel_stride), dtype=torch.int32, device=self.dev)
        self.sel_cnt = torch.empty((B, self.n_ret), dtype=torch.int32, device=self.dev)
        self.sel_mass = torch.empty((B, self.n_ret), dtype=torch.float32, device=self.dev)
        self.sel_thr = torch.empty((B, self.n_ret), dtype=torch.float32, device=self.dev)
        self.sel_tie = torch.empty((B, self.n_ret), dtype=torch.int32, device=self.dev)
        self.out = torch.empty((B, self.Hq, 128), dtype=torch.bfloat16, device=self.dev)
        self.lse = torch.empty((B, self.Hq), dtype=torch.float32, device=self.dev)
        # local heads do not depend on the retrieval heads: their attention runs on a second stream with a workspace
        # of its own and joins before the step returns
        self.side = torch.cuda.Stream(device=self.dev)
        self.workspace_local = torch.empty_like(self.workspace)
        self.has_local = len(data.heads.local_kv_heads) > 0

    def build_index_cache(self, step: int = 1 << 17):
        for b in range(self.B):
            for lo in range(0, self.L, step):
                self.index_keys_range(b, lo, min(self.L, lo + step))

    def step(self, q, k_pre_new):
        """q: bf16 [B, Hq, 128]; k_pre_new: bf16 [B, n_index_heads, 128] pre-RoPE keys of the newest tokens."""
        d, p = self.data, self.params
        main = torch.cuda.current_stream()
        if self.has_local:
            self.side.wait_stream(main)
            rb.rtp_local_attn(self.ctx, p, self.cache, q, d.row_seq, d.row_pos, 0, 0, self.B, self.out, self.lse,
                              self.workspace_local, self.status, stream=self.side)
        rb.rtp_index_keys(self.ctx, p, self.cache, k_pre_new, d.w_k, d.row_seq, d.row_pos)
        rb.rtp_topp_select(self.ctx, p, self.cache, q, d.w_q, d.row_seq, d.row_pos, 0, 0, self.B, self.sel_idx,
                           self.sel_cnt, self.sel_mass, self.sel_thr, self.sel_tie, self.status, self.workspace)
        rb.rtp_sparse_attn_decode(self.ctx, p, self.cache, q, d.row_seq, d.row_pos, self.sel_idx, self.sel_cnt,
                                  self.out, self.lse, self.workspace, self.status)
        if self.has_local:
            main.wait_stream(self.side)

    def step_blocks(self, q, k_pre_new):
        """The same decode step with the block-wise selector of Section 3.4: whole 64-key pages are selected by their
        log-sum-exp mass and attended to.  Buffers are made on first use."""
        d, p = self.data, self.params
        if not hasattr(self, "blk_idx"):
            n_b = (self.L + 63) // 64
            self.blk_idx = torch.empty((self.B, self.n_ret, n_b), dtype=torch.int32, device=self.dev)
            self.blk_cnt = torch.empty((self.B, self.n_ret), dtype=torch.int32, device=self.dev)
            self.blk_ws = torch.empty(max(1 << 16, rb.rtp_block_workspace_bytes(p, self.B, self.L)), dtype=torch.uint8,
                                      device=self.dev)
        main = torch.cuda.current_stream()
        if self.has_local:
            self.side.wait_stream(main)
            rb.rtp_local_attn(self.ctx, p, self.cache, q, d.row_seq, d.row_pos, 0, 0, self.B, self.out, self.lse,
                              self.workspace_local, self.status, stream=self.side)
        rb.rtp_index_keys(self.ctx, p, self.cache, k_pre_new, d.w_k, d.row_seq, d.row_pos)
        rb.rtp_topp_select_blocks_rows(self.ctx, p, self.cache, q, d.w_q, d.row_seq, d.row_pos, self.blk_idx, self.blk_cnt,
                                       self.sel_mass, self.sel_thr, self.sel_tie, self.status, self.blk_ws)
        rb.rtp_sparse_attn_decode_blocks(self.ctx, p, self.cache, q, d.row_seq, d.row_pos, self.blk_idx, self.blk_cnt,
                                         self.out, self.lse, self.workspace, self.status)
        if self.has_local:
            main.wait_stream(self.side)

    def step_dense(self, q):
        d = self.data
        rb.rtp_dense_attn_decode(self.ctx, self.params, self.cache, q, d.row_seq, d.row_pos, None, self.out, self.lse,
                                 self.workspace, self.status)
