"""Thin ctypes binding of the C ABI in ``include/rtp.h``.

Argument marshalling only: every step of the path runs inside ``librtp.so``.
Tensors are torch CUDA tensors (torch is used for device memory and streams);
bf16 tensors may be ``torch.bfloat16`` or raw ``int16``/``uint16`` views.  There
is no CPU fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_LIB: Optional[C.CDLL] = None
_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "librtp.so")

RTP_OK, RTP_ERR_INVALID, RTP_ERR_CAPACITY, RTP_ERR_UNSUPPORTED, RTP_ERR_CUDA, RTP_ERR_TIMEOUT = range(6)
RTP_IKEY_BF16, RTP_IKEY_E4M3 = 0, 1
_STATUS_NAMES = ["RTP_OK", "RTP_ERR_INVALID", "RTP_ERR_CAPACITY", "RTP_ERR_UNSUPPORTED", "RTP_ERR_CUDA",
                 "RTP_ERR_TIMEOUT"]

EXPORTS = [
    "rtp_version", "rtp_struct_bytes", "rtp_create", "rtp_destroy", "rtp_last_error", "rtp_debug_wait_test", "rtp_debug_select_path", "rtp_workspace_bytes", "rtp_check_status",
    "rtp_kv_append", "rtp_index_keys", "rtp_index_queries", "rtp_index_score", "rtp_topp_select", "rtp_sparse_attn_decode", "rtp_sparse_attn_decode_static",
    "rtp_sparse_attn_prefill", "rtp_local_attn", "rtp_dense_attn_prefill", "rtp_dense_attn_decode",
    "rtp_block_workspace_bytes", "rtp_topp_select_blocks", "rtp_sparse_attn_prefill_blocks",
    "rtp_topp_select_blocks_rows", "rtp_sparse_attn_decode_blocks",
]


class RtpError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        name = _STATUS_NAMES[code] if 0 <= code < len(_STATUS_NAMES) else str(code)
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


class RtpParams(C.Structure):
    _fields_ = [
        ("head_dim", C.c_int32), ("index_dim", C.c_int32), ("page_size", C.c_int32),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("n_index_heads", C.c_int32),
        ("n_ret_q_heads", C.c_int32), ("n_local_kv_heads", C.c_int32),
        ("n_sink", C.c_int32), ("window", C.c_int32),
        ("top_p", C.c_float), ("score_scale", C.c_float), ("sm_scale", C.c_float),
        ("ret_q_heads", C.POINTER(C.c_int32)), ("q_head_to_index_head", C.POINTER(C.c_int32)),
        ("index_head_kv", C.POINTER(C.c_int32)), ("local_kv_heads", C.POINTER(C.c_int32)),
        ("top_k", C.c_int32), ("force_sink", C.c_int32), ("force_recent", C.c_int32),
    ]


class RtpCache(C.Structure):
    _fields_ = [
        ("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("ikey_pages", C.c_void_p),
        ("block_table", C.c_void_p), ("seq_lens", C.c_void_p),
        ("num_pages", C.c_int32), ("batch", C.c_int32), ("max_pages", C.c_int32),
        ("k_local_pages", C.c_void_p), ("v_local_pages", C.c_void_p), ("local_block_table", C.c_void_p),
        ("n_local_pages", C.c_int32), ("sink_pages", C.c_int32), ("ring_pages", C.c_int32),
        ("ikey_format", C.c_int32),
    ]


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads ``librtp.so`` (built in-tree by ``build.py``); raises if it is missing."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RtpError(RTP_ERR_CUDA, "load_library",
                       f"{p} not found: build it with `python -m paper_2605_16928_b200.build`")
    lib = C.CDLL(p)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    PP, PC = C.POINTER(RtpParams), C.POINTER(RtpCache)
    lib.rtp_version.restype = i32
    lib.rtp_version.argtypes = []
    lib.rtp_struct_bytes.restype = sz
    lib.rtp_struct_bytes.argtypes = [i32]
    if lib.rtp_struct_bytes(0) != C.sizeof(RtpParams) or lib.rtp_struct_bytes(1) != C.sizeof(RtpCache):
        raise RtpError(RTP_ERR_INVALID, "load_library",
                       "the binding's argument blocks do not have the library's layout (rebuild the library)")
    lib.rtp_create.restype = i32
    lib.rtp_create.argtypes = [C.POINTER(vp)]
    lib.rtp_destroy.restype = None
    lib.rtp_destroy.argtypes = [vp]
    lib.rtp_last_error.restype = C.c_char_p
    lib.rtp_last_error.argtypes = [vp]
    lib.rtp_debug_wait_test.restype = i32
    lib.rtp_debug_wait_test.argtypes = [vp, i64, i32]
    lib.rtp_debug_select_path.restype = i32
    lib.rtp_debug_select_path.argtypes = [vp, i32]
    lib.rtp_workspace_bytes.restype = sz
    lib.rtp_workspace_bytes.argtypes = [PP, i64, i64]
    lib.rtp_check_status.restype = i32
    lib.rtp_check_status.argtypes = [vp, vp, vp]
    lib.rtp_index_keys.restype = i32
    lib.rtp_index_keys.argtypes = [vp, PP, PC, vp, vp, vp, vp, i64, vp]
    lib.rtp_kv_append.restype = i32
    lib.rtp_kv_append.argtypes = [vp, PP, PC, vp, vp, vp, vp, i64, vp, vp]
    lib.rtp_index_queries.restype = i32
    lib.rtp_index_queries.argtypes = [vp, PP, vp, vp, i64, vp, vp]
    lib.rtp_index_score.restype = i32
    lib.rtp_index_score.argtypes = [vp, PP, PC, vp, vp, vp, vp, i64, vp, i64, vp, vp, vp, sz, vp, vp]
    lib.rtp_topp_select.restype = i32
    lib.rtp_topp_select.argtypes = [vp, PP, PC, vp, vp, vp, vp, i32, i32, i64, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.rtp_sparse_attn_decode.restype = i32
    lib.rtp_sparse_attn_decode.argtypes = [vp, PP, PC, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, sz, vp, vp]
    lib.rtp_sparse_attn_decode_static.restype = i32
    lib.rtp_sparse_attn_decode_static.argtypes = [vp, PP, PC, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, vp]
    lib.rtp_sparse_attn_prefill.restype = i32
    lib.rtp_sparse_attn_prefill.argtypes = [vp, PP, PC, vp, vp, vp, i32, i32, i64, vp, i64, vp, vp, vp, vp, vp, vp,
                                            sz, vp, vp]
    lib.rtp_block_workspace_bytes.restype = sz
    lib.rtp_block_workspace_bytes.argtypes = [PP, i64, i64]
    lib.rtp_topp_select_blocks.restype = i32
    lib.rtp_topp_select_blocks.argtypes = [vp, PP, PC, vp, vp, i32, i32, i64, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.rtp_sparse_attn_prefill_blocks.restype = i32
    lib.rtp_sparse_attn_prefill_blocks.argtypes = [vp, PP, PC, vp, i32, i32, i64, vp, i64, vp, vp, vp, vp]
    lib.rtp_topp_select_blocks_rows.restype = i32
    lib.rtp_topp_select_blocks_rows.argtypes = [vp, PP, PC, vp, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.rtp_sparse_attn_decode_blocks.restype = i32
    lib.rtp_sparse_attn_decode_blocks.argtypes = [vp, PP, PC, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, sz, vp, vp]
    lib.rtp_local_attn.restype = i32
    lib.rtp_local_attn.argtypes = [vp, PP, PC, vp, vp, vp, i32, i32, i64, vp, vp, vp, sz, vp, vp]
    lib.rtp_dense_attn_prefill.restype = i32
    lib.rtp_dense_attn_prefill.argtypes = [vp, PP, PC, vp, i32, i32, i64, vp, i32, vp, vp, vp, vp]
    lib.rtp_dense_attn_decode.restype = i32
    lib.rtp_dense_attn_decode.argtypes = [vp, PP, PC, vp, vp, vp, i64, vp, i32, vp, vp, vp, sz, vp, vp]
    if path is None:
        _LIB = lib
    return lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream) or None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None


def _i32_array(vals: Sequence[int]):
    arr = (C.c_int32 * max(1, len(vals)))(*[int(v) for v in vals])
    return arr


class Params:
    """Owns an ``rtp_params`` block and the host head-map arrays it points to."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, ret_q_heads: Sequence[int],
                 q_head_to_index_head: Sequence[int], index_head_kv: Sequence[int],
                 local_kv_heads: Sequence[int], n_sink: int = 4, window: int = 8192, top_p: float = 0.9,
                 score_scale: float = 1.0, sm_scale: float = 128 ** -0.5, top_k: int = 0, force_sink: int = 0,
                 force_recent: int = 0):
        self._a = _i32_array(ret_q_heads)
        self._b = _i32_array(q_head_to_index_head)
        self._c = _i32_array(index_head_kv)
        self._d = _i32_array(local_kv_heads)
        self.n_ret = len(ret_q_heads)
        self.n_q_heads = n_q_heads
        self.n_kv_heads = n_kv_heads
        self.n_index_heads = len(index_head_kv)
        self.ret_q_heads = list(ret_q_heads)
        self.local_kv_heads = list(local_kv_heads)
        self.c = RtpParams(128, 16, 64, n_q_heads, n_kv_heads, len(index_head_kv), len(ret_q_heads),
                           len(local_kv_heads), n_sink, window, top_p, score_scale, sm_scale,
                           C.cast(self._a, C.POINTER(C.c_int32)), C.cast(self._b, C.POINTER(C.c_int32)),
                           C.cast(self._c, C.POINTER(C.c_int32)), C.cast(self._d, C.POINTER(C.c_int32)),
                           top_k, force_sink, force_recent)

    @classmethod
    def from_workload(cls, wl, **over) -> "Params":
        h = wl.heads
        kw = dict(n_q_heads=h.n_q_heads, n_kv_heads=h.n_kv_heads, ret_q_heads=h.ret_q_heads,
                  q_head_to_index_head=h.q_head_to_index_head, index_head_kv=h.index_head_kv,
                  local_kv_heads=h.local_kv_heads, n_sink=h.n_sink, window=h.window, top_p=wl.top_p,
                  score_scale=wl.score_scale, sm_scale=wl.sm_scale)
        kw.update(over)
        return cls(**kw)

    def ref(self):
        return C.byref(self.c)


def make_cache(k_pages, v_pages, ikey_pages, block_table, seq_lens, k_local_pages=None, v_local_pages=None,
               local_block_table=None, sink_pages: int = 0, ikey_format: Optional[int] = None) -> RtpCache:
    """Describes caller-owned paged caches (torch CUDA tensors) to the library.  With ``k_local_pages`` the cache is
    truncated for local heads: ``k_pages`` / ``v_pages`` hold the other KV heads only, the local heads live in the
    local pool behind ``local_block_table`` [batch, sink_pages + ring_pages]."""
    num_pages = int((k_pages if k_pages is not None else ikey_pages).shape[0])
    if ikey_format is None:   # the tensor's element size says which: uint8 pages are E4M3 codes
        ikey_format = RTP_IKEY_E4M3 if (ikey_pages is not None and ikey_pages.element_size() == 1) else RTP_IKEY_BF16
    n_local, ring = 0, 0
    if k_local_pages is not None:
        n_local = int(k_local_pages.shape[0])
        ring = int(local_block_table.shape[1]) - int(sink_pages)
    return RtpCache(_ptr(k_pages), _ptr(v_pages), _ptr(ikey_pages), _ptr(block_table), _ptr(seq_lens),
                    num_pages, int(block_table.shape[0]), int(block_table.shape[1]),
                    _ptr(k_local_pages), _ptr(v_local_pages), _ptr(local_block_table), n_local, int(sink_pages), ring,
                    int(ikey_format))


class Context:
    """``rtp_ctx`` for the current CUDA device."""

    def __init__(self):
        self.lib = load_library()
        h = C.c_void_p()
        rc = self.lib.rtp_create(C.byref(h))
        if rc != RTP_OK:
            raise RtpError(rc, "rtp_create", "needs a CUDA device of compute capability 10.x")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.rtp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != RTP_OK:
            raise RtpError(rc, where, (self.lib.rtp_last_error(self.h) or b"").decode())


def rtp_debug_select_path(ctx: Context, path: int):
    """0: the decode selection picks its implementation by size; 1: always the general (multi-kernel) path."""
    ctx._check(ctx.lib.rtp_debug_select_path(ctx.h, int(path)), "rtp_debug_select_path")


def rtp_debug_wait_test(ctx: Context, wait_limit_ns: int, drop_first_key_signal: bool):
    ctx._check(ctx.lib.rtp_debug_wait_test(ctx.h, int(wait_limit_ns), 1 if drop_first_key_signal else 0),
               "rtp_debug_wait_test")


def rtp_version() -> int:
    return int(load_library().rtp_version())


def rtp_workspace_bytes(params: Params, rows: int, max_seq_len: int) -> int:
    return int(load_library().rtp_workspace_bytes(params.ref(), rows, max_seq_len))


def rtp_check_status(ctx: Context, status, stream=None) -> int:
    return int(ctx.lib.rtp_check_status(ctx.h, _ptr(status), _stream(stream)))


def rtp_index_keys(ctx, params, cache, k_pre, w_k, tok_seq, tok_pos, stream=None):
    ctx._check(ctx.lib.rtp_index_keys(ctx.h, params.ref(), C.byref(cache), _ptr(k_pre), _ptr(w_k), _ptr(tok_seq),
                                      _ptr(tok_pos), int(tok_seq.shape[0]), _stream(stream)), "rtp_index_keys")


def rtp_kv_append(ctx, params, cache, k_new, v_new, tok_seq, tok_pos, status, stream=None):
    ctx._check(ctx.lib.rtp_kv_append(ctx.h, params.ref(), C.byref(cache), _ptr(k_new), _ptr(v_new), _ptr(tok_seq),
                                     _ptr(tok_pos), int(tok_seq.shape[0]), _ptr(status), _stream(stream)),
               "rtp_kv_append")


def rtp_index_queries(ctx, params, q_pre, w_q, qt_out, stream=None):
    ctx._check(ctx.lib.rtp_index_queries(ctx.h, params.ref(), _ptr(q_pre), _ptr(w_q), int(q_pre.shape[0]),
                                         _ptr(qt_out), _stream(stream)), "rtp_index_queries")


def rtp_index_score(ctx, params, cache, q_pre, w_q, row_seq, row_pos, scores_out, row_max_out, row_sum_out,
                    workspace, status, stream=None):
    stride = int(scores_out.shape[-1]) if scores_out is not None else 0
    ctx._check(ctx.lib.rtp_index_score(ctx.h, params.ref(), C.byref(cache), _ptr(q_pre), _ptr(w_q), _ptr(row_seq),
                                       _ptr(row_pos), int(row_seq.shape[0]), _ptr(scores_out), stride,
                                       _ptr(row_max_out), _ptr(row_sum_out), _ptr(workspace),
                                       int(workspace.numel() * workspace.element_size()), _ptr(status),
                                       _stream(stream)), "rtp_index_score")


def rtp_topp_select(ctx, params, cache, q_pre, w_q, row_seq, row_pos, seq_id, q_start, n_rows, sel_idx, sel_count,
                    sel_mass, sel_thresh, sel_tie_last, status, workspace, stream=None):
    stride = int(sel_idx.shape[-1]) if sel_idx is not None else 0
    ctx._check(ctx.lib.rtp_topp_select(ctx.h, params.ref(), C.byref(cache), _ptr(q_pre), _ptr(w_q), _ptr(row_seq),
                                       _ptr(row_pos), int(seq_id), int(q_start), int(n_rows), _ptr(sel_idx), stride,
                                       _ptr(sel_count), _ptr(sel_mass), _ptr(sel_thresh), _ptr(sel_tie_last),
                                       _ptr(status), _ptr(workspace),
                                       int(workspace.numel() * workspace.element_size()), _stream(stream)),
               "rtp_topp_select")


def rtp_sparse_attn_decode(ctx, params, cache, q, row_seq, row_pos, sel_idx, sel_count, out, lse, workspace, status,
                           stream=None):
    ctx._check(ctx.lib.rtp_sparse_attn_decode(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(row_seq),
                                              _ptr(row_pos), int(row_seq.shape[0]), _ptr(sel_idx),
                                              int(sel_idx.shape[-1]), _ptr(sel_count), _ptr(out), _ptr(lse),
                                              _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                              _ptr(status), _stream(stream)), "rtp_sparse_attn_decode")


def rtp_sparse_attn_decode_static(ctx, params, cache, q, row_seq, row_pos, sel_idx, sel_count, out, lse, status,
                                  stream=None):
    """rtp_sparse_attn_decode for callers that cannot hand over scratch memory: the split partials go to a
    512 KiB array built into the library, so nothing is allocated.  Calls must not overlap on the GPU."""
    ctx._check(ctx.lib.rtp_sparse_attn_decode_static(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(row_seq),
                                                     _ptr(row_pos), int(row_seq.shape[0]), _ptr(sel_idx),
                                                     int(sel_idx.shape[-1]), _ptr(sel_count), _ptr(out), _ptr(lse),
                                                     _ptr(status), _stream(stream)),
               "rtp_sparse_attn_decode_static")


def rtp_sparse_attn_prefill(ctx, params, cache, q, q_pre, w_q, seq_id, q_start, n_rows, sel_idx, sel_count,
                            sel_thresh, sel_tie_last, out, lse, workspace, status, stream=None):
    stride = int(sel_idx.shape[-1]) if sel_idx is not None else 0
    ctx._check(ctx.lib.rtp_sparse_attn_prefill(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(q_pre), _ptr(w_q),
                                               int(seq_id), int(q_start), int(n_rows), _ptr(sel_idx), stride,
                                               _ptr(sel_count), _ptr(sel_thresh), _ptr(sel_tie_last), _ptr(out),
                                               _ptr(lse), _ptr(workspace),
                                               int(workspace.numel() * workspace.element_size()), _ptr(status),
                                               _stream(stream)), "rtp_sparse_attn_prefill")


def rtp_block_workspace_bytes(params: Params, rows: int, max_seq_len: int) -> int:
    return int(load_library().rtp_block_workspace_bytes(params.ref(), rows, max_seq_len))


def rtp_topp_select_blocks(ctx, params, cache, q_pre, w_q, seq_id, q_start, n_rows, block_mask, sel_count, sel_mass,
                           sel_thresh, sel_tie_last, status, workspace, stream=None):
    """block_mask: int32 / uint32 tensor [n_rows, n_ret, mask_words]."""
    ctx._check(ctx.lib.rtp_topp_select_blocks(ctx.h, params.ref(), C.byref(cache), _ptr(q_pre), _ptr(w_q), int(seq_id),
                                              int(q_start), int(n_rows), _ptr(block_mask), int(block_mask.shape[-1]),
                                              _ptr(sel_count), _ptr(sel_mass), _ptr(sel_thresh), _ptr(sel_tie_last),
                                              _ptr(status), _ptr(workspace),
                                              int(workspace.numel() * workspace.element_size()), _stream(stream)),
               "rtp_topp_select_blocks")


def rtp_topp_select_blocks_rows(ctx, params, cache, q_pre, w_q, row_seq, row_pos, block_idx, sel_count, sel_mass,
                                sel_thresh, sel_tie_last, status, workspace, stream=None):
    """block_idx: int32 tensor [R, n_ret, block_stride] of logical page numbers (or None: counts only)."""
    stride = int(block_idx.shape[-1]) if block_idx is not None else 0
    ctx._check(ctx.lib.rtp_topp_select_blocks_rows(ctx.h, params.ref(), C.byref(cache), _ptr(q_pre), _ptr(w_q),
                                                   _ptr(row_seq), _ptr(row_pos), int(row_seq.shape[0]),
                                                   _ptr(block_idx), stride, _ptr(sel_count), _ptr(sel_mass),
                                                   _ptr(sel_thresh), _ptr(sel_tie_last), _ptr(status), _ptr(workspace),
                                                   int(workspace.numel() * workspace.element_size()), _stream(stream)),
               "rtp_topp_select_blocks_rows")


def rtp_sparse_attn_decode_blocks(ctx, params, cache, q, row_seq, row_pos, block_idx, block_count, out, lse, workspace,
                                  status, stream=None):
    ctx._check(ctx.lib.rtp_sparse_attn_decode_blocks(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(row_seq),
                                                     _ptr(row_pos), int(row_seq.shape[0]), _ptr(block_idx),
                                                     int(block_idx.shape[-1]), _ptr(block_count), _ptr(out), _ptr(lse),
                                                     _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                                     _ptr(status), _stream(stream)), "rtp_sparse_attn_decode_blocks")


def rtp_sparse_attn_prefill_blocks(ctx, params, cache, q, seq_id, q_start, n_rows, block_mask, out, lse, status,
                                   stream=None):
    ctx._check(ctx.lib.rtp_sparse_attn_prefill_blocks(ctx.h, params.ref(), C.byref(cache), _ptr(q), int(seq_id),
                                                      int(q_start), int(n_rows), _ptr(block_mask),
                                                      int(block_mask.shape[-1]), _ptr(out), _ptr(lse), _ptr(status),
                                                      _stream(stream)), "rtp_sparse_attn_prefill_blocks")


def rtp_local_attn(ctx, params, cache, q, row_seq, row_pos, seq_id, q_start, n_rows, out, lse, workspace, status,
                   stream=None):
    ws_bytes = int(workspace.numel() * workspace.element_size()) if workspace is not None else 0
    ctx._check(ctx.lib.rtp_local_attn(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(row_seq), _ptr(row_pos),
                                      int(seq_id), int(q_start), int(n_rows), _ptr(out), _ptr(lse), _ptr(workspace),
                                      ws_bytes, _ptr(status), _stream(stream)), "rtp_local_attn")


def rtp_dense_attn_prefill(ctx, params, cache, q, seq_id, q_start, n_rows, kv_heads, out, lse, status, stream=None):
    arr = _i32_array(kv_heads) if kv_heads is not None else None
    ctx._check(ctx.lib.rtp_dense_attn_prefill(ctx.h, params.ref(), C.byref(cache), _ptr(q), int(seq_id), int(q_start),
                                              int(n_rows), C.cast(arr, C.c_void_p) if arr is not None else None,
                                              len(kv_heads) if kv_heads is not None else 0, _ptr(out), _ptr(lse),
                                              _ptr(status), _stream(stream)), "rtp_dense_attn_prefill")


def rtp_dense_attn_decode(ctx, params, cache, q, row_seq, row_pos, kv_heads, out, lse, workspace, status,
                          stream=None):
    arr = _i32_array(kv_heads) if kv_heads is not None else None
    ctx._check(ctx.lib.rtp_dense_attn_decode(ctx.h, params.ref(), C.byref(cache), _ptr(q), _ptr(row_seq),
                                             _ptr(row_pos), int(row_seq.shape[0]),
                                             C.cast(arr, C.c_void_p) if arr is not None else None,
                                             len(kv_heads) if kv_heads is not None else 0, _ptr(out), _ptr(lse),
                                             _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                             _ptr(status), _stream(stream)), "rtp_dense_attn_decode")
