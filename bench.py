#!/usr/bin/env python
"""Benchmark of the sparse-attention hot path on B200.

Default workload ("c3"): chunked prefill of one 128K-token sequence (32 query / 8 KV heads, 2 retrieval
KV heads with a 16-dim indexer and top-p 0.9, 6 local heads with 4 sinks + 8192 window, chunk 8192).
One step = the whole hot path over the sequence: per chunk, index-key projection and append, fused
indexer + top-p thresholds, threshold-masked sparse attention on retrieval heads and sink+window
attention on local heads.  Metric: prefill tokens per second.

The JSON line also carries the dense in-library baseline, decode-step latencies (sparse path vs dense
split-KV decode), the roofline of the dominant kernel and the CPU oracle timed on the host cores.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c3|c4|c5]

--workload c4 is the one-million-token prefill with planted needles (chunk 16K, one retrieval KV head);
--workload c5 is the long-context decode sweep (batch x context x top-p x score temperature) printed as one table.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"],
                                     parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm)); out["sm_max_mhz"] = float(max(mx)); out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


def ev_time_ms(fn, stream):
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream); fn(); e1.record(stream); e1.synchronize()
    return e0.elapsed_time(e1)


# ------------------------------------------------------------------------------------------------ prefill
def prefill_tile_flops(L: int, chunk: int, group: int, n_kv_heads: int, mode: str, n_sink: int, window: int,
                       tile_keys: int = 128) -> float:
    """FLOPs of the key tiles a prefill kernel visits: 128 MMA rows x tile_keys keys x 128 dims x (QK^T + PV).
    The tcgen05 kernel (dense, sink+window, sparse) walks 128-key tiles; the warp-MMA fallback 64-key tiles."""
    bmp = 128 // group
    per_tile = 128 * tile_keys * 128 * 2 * 2
    tiles = 0
    for q_start in range(0, L, chunk):
        C = min(chunk, L - q_start)
        for r0 in range(0, C, bmp):
            m0 = q_start + r0
            m_last = m0 + min(bmp, C - r0) - 1
            kt_last = m_last // tile_keys
            if mode == "local":
                kt_first = max(0, m0 - window + 1) // tile_keys
                tiles += min((n_sink + tile_keys - 1) // tile_keys, kt_first) + kt_last - kt_first + 1
            else:
                tiles += kt_last + 1
    return float(tiles) * per_tile * n_kv_heads


def bench_prefill(args, rank, world, device):
    import torch
    from paper_2605_16928_b200 import synth_device, pipeline
    c4 = args.workload == "c4"
    L, chunk = args.seq_len or (1048576 if c4 else 131072), args.chunk or (16384 if c4 else 8192)
    if c4:
        data = synth_device.config_4_device(L=L, device=device)
    else:
        data = synth_device.config_3_device(L=L, device=device)
    path = pipeline.PrefillPath(data, chunk)
    stream = torch.cuda.current_stream()
    out = torch.empty((L, path.Hq, 128), dtype=torch.bfloat16, device=device)
    k_pre = data.k_pre_rows(0, 0, L)
    chunks = path.chunks()

    def step():
        if args.path == "blocks":
            for (s, C) in chunks:
                path.run_chunk_blocks(s, C, data.q[s:s + C], k_pre[s:s + C], out[s:s + C])
            return
        for (s, C) in chunks:
            path.run_chunk(s, C, data.q[s:s + C], k_pre[s:s + C], out[s:s + C])

    def step_dense():
        for (s, C) in chunks:
            path.run_chunk_dense(s, C, data.q[s:s + C], out[s:s + C])

    return data, path, step, step_dense, out, k_pre, chunks, L, chunk, stream


def prefill_sparsity(path, data, chunks, L, rows_per_chunk=16, n_chunks=4):
    """Compute sparsity (per query head) and memory sparsity (union over the query heads of a KV head) of the retrieval
    heads (Section 3.2), counted on sampled rows of a few chunks from the selection the library wrote and the scores it
    materialises for those rows.  Counting only: no part of the timed path."""
    import torch
    from paper_2605_16928_b200 import binding as rb
    g, n_ret = data.heads.group, path.n_ret
    pick = sorted({int(round(x)) for x in np.linspace(0, len(chunks) - 1, min(n_chunks, len(chunks)))})
    rng = np.random.default_rng(7)
    comp, mem, ratio = [], [], []
    R = rows_per_chunk
    sc = torch.empty((R, n_ret, L), dtype=torch.float32, device=path.dev)
    ws = torch.empty(rb.rtp_workspace_bytes(path.params, R, L), dtype=torch.uint8, device=path.dev)
    pos = torch.arange(L, device=path.dev)
    for ci in pick:
        s0, C = chunks[ci]
        q = data.q[s0:s0 + C]
        rb.rtp_topp_select(path.ctx, path.params, path.cache, q, data.w_q, None, None, 0, s0, C, None, path.sel_cnt,
                           path.sel_mass, path.sel_thr, path.sel_tie, path.status, path.workspace)
        r = torch.from_numpy(np.sort(rng.choice(C, size=min(R, C), replace=False))).to(path.dev)
        rows = (r + s0).to(torch.int32)
        sc.fill_(float("nan"))
        rb.rtp_index_score(path.ctx, path.params, path.cache, q[r].contiguous(), data.w_q,
                           torch.zeros(len(r), dtype=torch.int32, device=path.dev), rows, sc[:len(r)], None, None, ws,
                           path.status)
        thr, tie = path.sel_thr[r][:, :, None], path.sel_tie[r][:, :, None]
        member = (sc[:len(r)] > thr) | ((sc[:len(r)] == thr) & (pos[None, None, :] <= tie))
        per_head = member.sum(-1).double()                                          # [R, n_ret]
        union = member.view(len(r), n_ret // g, g, L).any(2).sum(-1).double()        # [R, n_ret / g]
        ctx_len = (rows.double() + 1.0)[:, None]
        comp.append((per_head / ctx_len).mean().item())
        mem.append((union / ctx_len).mean().item())
        ratio.append((union / per_head.view(len(r), n_ret // g, g).mean(-1)).mean().item())
    return {"compute_sparsity": 1.0 - float(np.mean(comp)), "memory_sparsity": 1.0 - float(np.mean(mem)),
            "union_over_mean_head_set": float(np.mean(ratio)),
            "sample": f"{R} rows in each of chunks {pick}; union over the {g} query heads of a retrieval KV head"}


def cpu_oracle_prefill(data, L, rows, budget_s=25.0):
    """Times the CPU oracle on a bounded sample of query rows of the prefill workload (all 32 heads)."""
    from oracle import rtp_oracle as orc
    heads = data.heads
    g = heads.group
    to_np = lambda t: t.contiguous().view(__import__("torch").int16).cpu().numpy().view(np.uint16)
    kv = {h: data.logical_kv(0, h, 0, L) for h in range(heads.n_kv_heads)}
    q = to_np(data.q[[int(r) for r in rows]])
    w_q, w_k = to_np(data.w_q), to_np(data.w_k)
    c0 = time.process_time()
    t0 = time.perf_counter()
    kt = [orc.index_project(kv[heads.index_head_kv[j]][0], w_k[j]) for j in range(heads.n_index_heads)]
    t_proj = time.perf_counter() - t0
    done, t_rows = 0, 0.0
    for k, m in enumerate(rows):
        t1 = time.perf_counter()
        for i, h in enumerate(heads.ret_q_heads):
            kh = h // g
            orc.retrieval_row(q[k, h], q[k, h], w_q[i], kt[heads.q_head_to_index_head[i]], kv[kh][0], kv[kh][1],
                              int(m), data.top_p, data.score_scale, data.sm_scale)
        for kh in heads.local_kv_heads:
            for j in range(g):
                orc.local_row(q[k, kh * g + j], kv[kh][0], kv[kh][1], int(m), heads.n_sink, heads.window, data.sm_scale)
        t_rows += time.perf_counter() - t1
        done += 1
        if t_rows + t_proj > budget_s:
            break
    per_tok = t_rows / done + t_proj / L
    # threads the oracle really kept busy: process CPU time over wall time (numpy's BLAS calls may use several, the
    # sorts and elementwise steps use one)
    busy = (time.process_time() - c0) / max(1e-9, t_rows + t_proj)
    return 1.0 / per_tok, done, t_rows + t_proj, max(1, int(round(busy)))


# ------------------------------------------------------------------------------------------------ decode extras
def bench_decode_point(device, name, L, B, top_p, frac, window, peaked_half, iters=20, variants=True):
    import torch
    from paper_2605_16928_b200 import synth_device, pipeline
    from paper_2605_16928_b200 import binding as rb
    data = synth_device.decode_device(L, B, top_p, frac, window, device=device, peaked_half=peaked_half, name=name)
    stride = int(min(L, max(4096, 4 * frac * L)))
    path = pipeline.DecodePath(data, stride)
    path.build_index_cache()
    k_pre_new = data.k_pre_rows(0, L - 1, L).repeat(B, 1, 1).contiguous()
    for b in range(B):
        k_pre_new[b] = data.k_pre_rows(b, L - 1, L)[0]
    stream = torch.cuda.current_stream()
    flush = torch.empty(192 << 20, dtype=torch.uint8, device=device)

    def timed(fn):
        for _ in range(3):
            fn()
        ts = []
        for _ in range(iters):
            flush.zero_()
            ts.append(ev_time_ms(fn, stream) * 1e3)
        return float(np.median(ts))

    def graph_timed(pth):
        """The same step replayed from a CUDA graph (the library calls captured once): no host launch cost."""
        try:
            graph = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=device)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                pth.step(data.q, k_pre_new)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            with torch.cuda.graph(graph):
                pth.step(data.q, k_pre_new)
            return timed(graph.replay)
        except Exception as exc:   # capture is an extra; the plain numbers stand on their own
            return f"not captured: {type(exc).__name__}"

    t_sparse = timed(lambda: path.step(data.q, k_pre_new))
    t_dense = timed(lambda: path.step_dense(data.q))
    t_graph = graph_timed(path)
    var = {}
    if variants:
        # the block-wise selector of Section 3.4 on the same data: 64-key pages chosen by log-sum-exp mass
        t_blk = timed(lambda: path.step_blocks(data.q, k_pre_new))
        blk_frac = float(path.blk_cnt.float().mean().item()) / ((L + 63) // 64)
        blk_status = path.status_code()
        path.step(data.q, k_pre_new)   # (the token-level outputs are what the figures below describe)
        torch.cuda.synchronize()
        # the fixed-budget variant the paper compares with (Section 4.1, k = 4096), same data and step
        path_k = pipeline.DecodePath(data, max(stride, 4096), top_k=4096)
        path_k.build_index_cache()
        t_topk = timed(lambda: path_k.step(data.q, k_pre_new))
        t_topk_graph = graph_timed(path_k)
        topk_status = path_k.status_code()
        del path_k
        # the 8-bit index-key cache (16 bytes per token and index head): same data, same step; how much of the bf16
        # selection it reproduces is reported beside the time
        path_8 = pipeline.DecodePath(data, stride, ikey_e4m3=True)
        path_8.build_index_cache()
        t_ikey8 = timed(lambda: path_8.step(data.q, k_pre_new))
        t_ikey8_graph = graph_timed(path_8)
        ikey8_status = path_8.status_code()
        inter = total = 0
        for b_ in range(min(B, 4)):
            for i_ in range(path.n_ret):
                s16 = path.sel_idx[b_, i_, : int(path.sel_cnt[b_, i_])]
                s8 = path_8.sel_idx[b_, i_, : int(path_8.sel_cnt[b_, i_])]
                inter += int(torch.isin(s8, s16).sum().item())
                total += int(s16.numel())
        ikey8_overlap = inter / max(1, total)
        # softmax mass, under the scores of the bf16 cache, of the sets chosen on the 8-bit cache (the target is top_p)
        nb = min(B, 4)
        sc16 = torch.empty((nb, path.n_ret, L), dtype=torch.float32, device=device)
        rb.rtp_index_score(path.ctx, path.params, path.cache, data.q[:nb].contiguous(), data.w_q, data.row_seq[:nb].contiguous(),
                           data.row_pos[:nb].contiguous(), sc16, None, None, path.workspace, path.status)
        masses = []
        for b_ in range(nb):
            for i_ in range(path.n_ret):
                row = sc16[b_, i_].double()
                w = torch.exp(row - row.max())
                ids8 = path_8.sel_idx[b_, i_, : int(path_8.sel_cnt[b_, i_])].long()
                masses.append(float((w[ids8].sum() / w.sum()).item()))
        del sc16
        ikey8_count_ratio = float(path_8.sel_cnt.float().mean().item()) / max(1.0, float(path.sel_cnt.float().mean().item()))
        del path_8
        var = {"block_topp_step_us": t_blk, "block_topp_selected_block_fraction": blk_frac, "block_topp_status": blk_status,
               "fixed_budget_4096_step_us": t_topk, "fixed_budget_4096_step_us_cuda_graph": t_topk_graph,
               "fixed_budget_status": topk_status,
               "ikey_e4m3_step_us": t_ikey8, "ikey_e4m3_step_us_cuda_graph": t_ikey8_graph, "ikey_e4m3_status": ikey8_status,
               "ikey_e4m3_share_of_bf16_set_kept": ikey8_overlap, "ikey_e4m3_count_ratio": ikey8_count_ratio,
               "ikey_e4m3_mass_under_bf16_scores": {"mean": float(np.mean(masses)), "min": float(np.min(masses))}}
    cnt = path.sel_cnt.float()
    n_ih = data.heads.n_index_heads
    sel_rows = float(cnt.sum().item())
    alg_bytes = B * n_ih * 32.0 * L + 512.0 * sel_rows + 8.0 * sel_rows + \
        B * len(data.heads.local_kv_heads) * 512.0 * min(L, 4 + window)
    res = {"workload": name, "batch": B, "context": L, "top_p": top_p,
           "selected_fraction_mean": float(cnt.mean().item()) / L,
           "sparse_step_us": t_sparse, "sparse_step_us_cuda_graph": t_graph, "dense_step_us": t_dense,
           "speedup_vs_dense": t_dense / t_sparse,
           **var,
           "algorithmic_bytes": alg_bytes, "sparse_path_gbs": alg_bytes / t_sparse / 1e3,
           "dense_gbs": B * data.heads.n_kv_heads * 512.0 * L / t_dense / 1e3,
           "status": path.status_code()}
    del path, data
    torch.cuda.empty_cache()
    return res


def bench_c5_sweep(device, iters=10, batches=(1, 4, 16), contexts=(131072, 524288, 1048576), tops=(0.8, 0.9, 0.99),
                   fracs=(0.001, 0.02, 0.2)):
    """The long-context decode sweep: one cache per (batch, context); top-p and the score temperature (set from the
    Gaussian closed form for a target selected fraction) change the queries only.  One row per point."""
    import torch
    from paper_2605_16928_b200 import synth_device, pipeline, binding as rb
    stream = torch.cuda.current_stream()
    flush = torch.empty(192 << 20, dtype=torch.uint8, device=device)

    def timed(fn):
        for _ in range(3):
            fn()
        ts = []
        for _ in range(iters):
            flush.zero_()
            ts.append(ev_time_ms(fn, stream) * 1e3)
        return float(np.median(ts))

    table = []
    for B in batches:
        for L in contexts:
            base = synth_device.decode_device(L, B, 0.9, 0.05, 4096, device=device)
            path = pipeline.DecodePath(base, L)
            path.build_index_cache()
            k_new = torch.stack([base.k_pre_rows(b, L - 1, L)[0] for b in range(B)]).contiguous()
            heads = base.heads
            g, n_ih, n_ret = heads.group, heads.n_index_heads, len(heads.ret_q_heads)
            t_dense = timed(lambda: path.step_dense(base.q))
            dense_bytes = B * heads.n_kv_heads * 512.0 * L
            for p in tops:
                for frac in fracs:
                    data = synth_device.decode_retarget(base, p, frac)
                    path.data, path.params = data, rb.Params.from_workload(data)
                    # the block-wise selector of Section 3.4 on the same point (64-key pages by log-sum-exp mass)
                    t_blk = timed(lambda: path.step_blocks(data.q, k_new))
                    blk_frac = float(path.blk_cnt.float().mean().item()) / ((L + 63) // 64)
                    blk_mass = float(path.sel_mass.mean().item())
                    t = timed(lambda: path.step(data.q, k_new))
                    cnt = path.sel_cnt.long()
                    # memory sparsity: union of the lists of the query heads that share a KV head
                    valid = torch.arange(L, device=device)[None, None, :] < cnt[:, :, None]
                    bi, hi, ji = torch.nonzero(valid, as_tuple=True)
                    mask = torch.zeros((B, n_ret // g, L), dtype=torch.bool, device=device)
                    mask[bi, hi // g, path.sel_idx[bi, hi, ji].long()] = True
                    union = mask.sum(-1).double()
                    del valid, bi, hi, ji, mask
                    sel_rows = float(cnt.sum().item())
                    alg = B * n_ih * 32.0 * L + 520.0 * sel_rows + B * len(heads.local_kv_heads) * 512.0 * min(L, 4 + 4096)
                    # K and V bytes held: every head in full, against retrieval heads in full + sink page and a ring of
                    # window / 64 + 2 pages for the local heads (the truncated cache layout of rtp_cache)
                    pages = (L + 63) // 64
                    kv_full = 2.0 * B * pages * heads.n_kv_heads * 16384
                    kv_trunc = 2.0 * B * (pages * (heads.n_kv_heads - len(heads.local_kv_heads)) +
                                          (1 + 4096 // 64 + 2) * len(heads.local_kv_heads)) * 16384
                    table.append({"batch": B, "context": L, "top_p": p, "target_fraction": frac,
                                  "kv_bytes_full": kv_full, "kv_bytes_truncated_local_heads": kv_trunc,
                                  "selected_fraction": sel_rows / (B * n_ret * L),
                                  "union_fraction_per_kv_head": float(union.mean().item()) / L,
                                  "sparse_step_us": t, "dense_step_us": t_dense, "speedup_vs_dense": t_dense / t,
                                  "block_topp_step_us": t_blk, "block_topp_selected_block_fraction": blk_frac,
                                  "block_topp_selected_mass": blk_mass,
                                  "algorithmic_bytes": alg, "sparse_path_gbs": alg / t / 1e3,
                                  "dense_gbs": dense_bytes / t_dense / 1e3, "status": path.status_code()})
            del path, base
            torch.cuda.empty_cache()
    return table


# ------------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c3", "c4", "c5"],
                    help="c3: 128K chunked prefill, 2 retrieval KV heads (default, the bench line); "
                         "c4: 1M prefill with planted needles, chunk 16K, 1 retrieval KV head (long run, no end-to-end "
                         "leg); c5: the long-context decode sweep as one table")
    ap.add_argument("--path", default="tokens", choices=["tokens", "blocks"],
                    help="selection used by the timed step: token-level top-p (default, the bench line) or the block-wise "
                         "top-p of the paper's kernel section (reported as block_topp_path in the default run)")
    ap.add_argument("--seq-len", type=int, default=0)
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--no-extras", action="store_true", help="skip the dense baseline, decode points and CPU oracle")
    ap.add_argument("--no-variants", action="store_true",
                    help="decode points: skip the fixed-budget and 8-bit index-key runs (used for ncu launch lists)")
    ap.add_argument("--decode-only", action="store_true",
                    help="run only the decode points (c2 and one c5 point) and print them; used for profiling")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    from paper_2605_16928_b200 import replicas
    rank, world, local_rank = replicas.env_rank_world()
    n_cores = len(os.sched_getaffinity(0))
    c4 = args.workload == "c4"
    L, chunk = args.seq_len or (1048576 if c4 else 131072), args.chunk or (16384 if c4 else 8192)
    config = {"workload": (f"c4_long_prefill_{L}" if c4 else
                           "c3_chunked_prefill_128k" if L == 131072 else f"c3_chunked_prefill_{L}"),
              "seq_len": L, "chunk": chunk, "n_q_heads": 32, "n_kv_heads": 8, "retrieval_kv_heads": 1 if c4 else 2,
              "index_dim": 16, "top_p": 0.9, "n_sink": 4, "window": 8192, "page_size": 64,
              "l2": "inputs_larger_than_l2", "parallelism": "replicas" if world > 1 else "single_gpu",
              "selection": "token-level top-p" if args.path == "tokens" else "block-wise top-p (64-key pages)"}

    if args.impl == "reference":
        # The reference arm is the CPU oracle, as it stands, on a bounded sample of the same workload.
        if rank != 0:
            return
        import torch
        from paper_2605_16928_b200 import synth_device
        dev = "cuda:0" if torch.cuda.is_available() else "cpu"
        data = synth_device.config_4_device(L=L, device=dev) if c4 else synth_device.config_3_device(L=L, device=dev)
        per_step = 24
        rows = np.linspace(L // 16, L - 1, 3 * per_step).astype(np.int64)
        vals = []
        t_all = time.perf_counter()
        for s in range(args.warmup + args.steps):
            v, done, _, used = cpu_oracle_prefill(data, L, rows[(s % 3)::3], budget_s=6.0)
            if s >= args.warmup:
                vals.append(v)
        value = float(np.mean(vals))
        line = {"impl": "reference", "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s",
                "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": 1e3 * L / value, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": used, "cores_available": n_cores,
                                 "kind": "oracle (numpy, fp64)",
                                 "sample": "up to 24 query rows x 32 heads per step (6 s budget), extrapolated to the sequence"},
                "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "wall_s": time.perf_counter() - t_all}
        print(json.dumps(line))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist = replicas.init("nccl", world)
    from paper_2605_16928_b200 import build as rbuild
    if rank == 0:
        rbuild.build_library()
    replicas.barrier(dist, device)
    peaks = load_peaks()

    if args.workload == "c5":
        if rank == 0:
            sampler = ClockSampler(local_rank)
            sampler.start()
            table = bench_c5_sweep(device, iters=max(3, args.steps))
            clocks = sampler.stop()
            ref = next(r for r in table if (r["batch"], r["context"], r["top_p"], r["target_fraction"]) == (4, 524288, 0.9, 0.02))
            hdr = f"{'B':>3} {'context':>8} {'p':>5} {'target':>7} {'selected':>9} {'union':>7} {'sparse us':>10} {'dense us':>10} {'x':>6} {'GB/s':>7} {'block us':>9} {'blocks':>7}"
            print(hdr, file=sys.stderr)
            for r in table:
                print(f"{r['batch']:>3} {r['context']:>8} {r['top_p']:>5} {r['target_fraction']:>7.3f} {r['selected_fraction']:>9.4f} "
                      f"{r['union_fraction_per_kv_head']:>7.4f} {r['sparse_step_us']:>10.1f} {r['dense_step_us']:>10.1f} "
                      f"{r['speedup_vs_dense']:>6.2f} {r['sparse_path_gbs']:>7.0f} {r['block_topp_step_us']:>9.1f} "
                      f"{r['block_topp_selected_block_fraction']:>7.4f}", file=sys.stderr)
            print(json.dumps({"metric": "decode_step_us", "value": ref["sparse_step_us"], "unit": "us", "n_gpus": 1,
                              "steps": max(3, args.steps), "warmup": 3, "ms_per_step": ref["sparse_step_us"] / 1e3,
                              "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                              "data": "synthetic", "clocks": clocks,
                              "config": {"workload": "c5_decode_sweep", "value_point": "batch 4, context 512K, top-p 0.9, target fraction 2 %",
                                         "l2": "flushed between timed iterations"},
                              "roofline": {"bound": "hbm", "achieved": ref["sparse_path_gbs"], "peak": peaks["hbm_gbs"],
                                           "unit": "GB/s", "frac": ref["sparse_path_gbs"] / peaks["hbm_gbs"], "traffic": None,
                                           "peak_source": peaks["source"]},
                              "table": table}))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    if args.decode_only:
        if rank == 0:
            dec = [bench_decode_point(device, "c2_decode_batched_gqa", 32768, 8, 0.95, 0.1, 2048, True, iters=max(3, args.steps), variants=not args.no_variants),
                   bench_decode_point(device, "c5_decode_b4_512k", 524288, 4, 0.9, 0.05, 4096, False, iters=max(3, args.steps), variants=not args.no_variants),
                   bench_decode_point(device, "c1_sized_decode_b1_4k", 4096, 1, 0.9, 0.05, 2048, False, iters=max(3, args.steps), variants=False)]
            print(json.dumps({"decode": dec}))
        return

    data, path, step, step_dense, out, k_pre, chunks, L, chunk, stream = bench_prefill(args, rank, world, device)

    def barrier():
        replicas.barrier(dist, device)

    # ---- device-resident timing ----
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    ms = replicas.max_over_ranks(dist, ms, device)
    ms_per_step = ms / args.steps
    value = replicas.whole_job_rate(world, L, ms_per_step)
    status = path.status_code()
    sel_frac = None if args.path == "blocks" else float((path.sel_cnt.float() / (path.pos_all[L - len(path.sel_cnt):].float()[:, None] + 1)).mean().item())

    from paper_2605_16928_b200 import binding as rb
    Hq, Hkv, nih = path.Hq, data.heads.n_kv_heads, data.heads.n_index_heads

    def run_e2e():
        # ---- end to end: pinned host buffers, H2D of the chunk's q / k / v / k_pre, D2H of its output ----
        h_q = torch.empty((L, Hq, 128), dtype=torch.bfloat16).pin_memory()
        h_q.copy_(data.q)
        h_kpre = torch.empty((L, nih, 128), dtype=torch.bfloat16).pin_memory()
        h_kpre.copy_(k_pre)
        h_k = torch.empty((L, Hkv, 128), dtype=torch.bfloat16).pin_memory()
        h_v = torch.empty((L, Hkv, 128), dtype=torch.bfloat16).pin_memory()
        for s in range(0, L, 16384):
            e = min(L, s + 16384)
            phys = data.block_table[0, s // 64:(e + 63) // 64].long()
            h_k[s:e].copy_(data.k_pages[phys].permute(0, 2, 1, 3).reshape(-1, Hkv, 128)[: e - s])
            h_v[s:e].copy_(data.v_pages[phys].permute(0, 2, 1, 3).reshape(-1, Hkv, 128)[: e - s])
        h_out = torch.empty((L, Hq, 128), dtype=torch.bfloat16).pin_memory()

        # Two sets of device staging buffers and a copy stream: the H2D copies of chunk i+1 and the D2H copy of chunk
        # i-1 overlap the kernels of chunk i (events order the hand-offs; everything ends on the compute stream).
        copy_stream = torch.cuda.Stream(device=device)
        stage = [dict(q=torch.empty((chunk, Hq, 128), dtype=torch.bfloat16, device=device),
                      kpre=torch.empty((chunk, nih, 128), dtype=torch.bfloat16, device=device),
                      k=torch.empty((chunk, Hkv, 128), dtype=torch.bfloat16, device=device),
                      v=torch.empty((chunk, Hkv, 128), dtype=torch.bfloat16, device=device),
                      out=torch.empty((chunk, Hq, 128), dtype=torch.bfloat16, device=device),
                      loaded=torch.cuda.Event(), computed=torch.cuda.Event(), drained=torch.cuda.Event()) for _ in range(2)]

        def step_e2e():
            copy_stream.wait_stream(stream)
            for b in stage:
                b["drained"].record(copy_stream)

            def load(i):
                s, C = chunks[i]
                b = stage[i & 1]
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(b["computed"])     # the previous user of this buffer set has finished computing
                    b["q"][:C].copy_(h_q[s:s + C], non_blocking=True)
                    b["kpre"][:C].copy_(h_kpre[s:s + C], non_blocking=True)
                    b["k"][:C].copy_(h_k[s:s + C], non_blocking=True)
                    b["v"][:C].copy_(h_v[s:s + C], non_blocking=True)
                    b["loaded"].record(copy_stream)

            for b in stage:
                b["computed"].record(stream)
            load(0)
            for i, (s, C) in enumerate(chunks):
                b = stage[i & 1]
                if i + 1 < len(chunks):
                    load(i + 1)
                stream.wait_event(b["loaded"])
                stream.wait_event(b["drained"])               # the output buffer of this set has been copied out
                rb.rtp_kv_append(path.ctx, path.params, path.cache, b["k"][:C], b["v"][:C], path.tok_seq[:C],
                                 path.pos_all[s:s + C], path.status)
                path.run_chunk(s, C, b["q"][:C], b["kpre"][:C], b["out"][:C])
                b["computed"].record(stream)
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(b["computed"])
                    h_out[s:s + C].copy_(b["out"][:C], non_blocking=True)
                    b["drained"].record(copy_stream)
            stream.wait_stream(copy_stream)

        step_e2e()
        barrier()
        n_e2e = max(1, min(args.steps, 3))
        e0.record(stream)
        for _ in range(n_e2e):
            step_e2e()
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1) / n_e2e
        ms_e2e = replicas.max_over_ranks(dist, ms_e2e, device)
        h2d = int(L * (Hq + 2 * Hkv + nih) * 128 * 2)
        d2h = int(L * Hq * 128 * 2)
        torch.cuda.synchronize()
        s_chk, C_chk = chunks[-1]
        step()                                                  # resident outputs for the comparison below
        torch.cuda.synchronize()
        e2e_ok = bool(torch.equal(h_out[s_chk:s_chk + C_chk].to(device), out[s_chk:s_chk + C_chk]))
        return ms_e2e, h2d, d2h, e2e_ok

    if args.workload == "c4" or args.path == "blocks":
        # 1M tokens: the pinned host copies of q and out alone are 17 GB; the end-to-end leg is run on c3's default path only
        ms_e2e, h2d, d2h, e2e_ok = None, 0, 0, None
    else:
        ms_e2e, h2d, d2h, e2e_ok = run_e2e()

    # ---- per-kernel timing of one instrumented step (not part of the timed region) ----
    klass = {"index_keys": 0.0, "select": 0.0, "sparse_attn": 0.0, "local_attn": 0.0}
    d, p = path.data, path.params
    n_selected = torch.zeros((), dtype=torch.float64, device=device)
    for (s, C) in chunks:
        q, kp, o = data.q[s:s + C], k_pre[s:s + C], out[s:s + C]
        klass["index_keys"] += ev_time_ms(lambda: rb.rtp_index_keys(path.ctx, p, path.cache, kp, d.w_k, path.tok_seq[:C], path.pos_all[s:s + C]), stream)
        klass["select"] += ev_time_ms(lambda: rb.rtp_topp_select(path.ctx, p, path.cache, q, d.w_q, None, None, 0, s, C, None, path.sel_cnt, path.sel_mass, path.sel_thr, path.sel_tie, path.status, path.workspace), stream)
        n_selected += path.sel_cnt[:C].sum(dtype=torch.float64)
        klass["sparse_attn"] += ev_time_ms(lambda: rb.rtp_sparse_attn_prefill(path.ctx, p, path.cache, q, q, d.w_q, 0, s, C, None, path.sel_cnt, path.sel_thr, path.sel_tie, o, None, path.workspace, path.status), stream)
        klass["local_attn"] += ev_time_ms(lambda: rb.rtp_local_attn(path.ctx, p, path.cache, q, None, None, 0, s, C, o, None, path.workspace, path.status), stream)
    g = data.heads.group
    fl_sparse = prefill_tile_flops(L, chunk, g, len(data.heads.ret_kv_heads), "dense", 4, 8192)
    fl_local = prefill_tile_flops(L, chunk, g, len(data.heads.local_kv_heads), "local", 4, 8192)
    fl_dense = prefill_tile_flops(L, chunk, g, data.heads.n_kv_heads, "dense", 4, 8192)
    pairs = sum((min(chunk, L - s)) * (2 * s + min(chunk, L - s) + 1) / 2 for s in range(0, L, chunk))
    dom = max(klass, key=klass.get)
    n_launch = len(chunks)
    if dom in ("sparse_attn", "local_attn"):
        fl = fl_sparse if dom == "sparse_attn" else fl_local
        achieved = fl / (klass[dom] * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        roofline = {"kernel": "attn_prefill_tc_kernel<sparse> (tcgen05)" if dom == "sparse_attn" else "attn_prefill_tc_kernel<local> (tcgen05)",
                    "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None, "peak_source": peaks["source"] + " (sustained bf16)",
                    "flops_per_launch": fl / n_launch, "launch_ms": klass[dom] / n_launch}
    else:
        # indexer + top-p: one exponential per score and pass on the special-function unit, the rest plain ALU work
        scores = pairs * len(data.heads.ret_q_heads)
        achieved = scores / (klass["select"] * 1e-3) / 1e12
        props = torch.cuda.get_device_properties(device)
        n_sm = props.multi_processor_count
        clk_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
        peak = 16.0 * n_sm * clk_mhz * 1e6 / 1e12
        alu_ops = 12.0
        peak_alu = n_sm * 128 * clk_mhz * 1e6 / alu_ops / 1e12
        roofline = {"kernel": "select_chunk_kernel", "bound": "alu", "achieved": achieved, "peak": peak,
                    "unit": "Tscore/s", "frac": achieved / peak, "traffic": None,
                    "peak_source": f"16 ex2 per clock per SM x {n_sm} SMs x {clk_mhz:.0f} MHz (median SM clock sampled in the timed region)",
                    "alu_derived": {"peak": peak_alu, "frac": achieved / peak_alu,
                                    "source": f"{n_sm} SMs x 128 lanes x {clk_mhz:.0f} MHz / {alu_ops:.0f} lane-ops per score and pass"},
                    "scores_per_launch": scores / n_launch, "launch_ms": klass["select"] / n_launch}
    useful_flops = float(n_selected.item()) * 128 * 2 * 2
    s6 = {"useful_flops": useful_flops, "executed_flops": fl_sparse, "union_factor": fl_sparse / max(1.0, useful_flops),
          "note": "executed = every causal 128-key tile of the retrieval heads (threshold-masked, no tile skipping); "
                  "useful = 512 flops per selected (row, head, key)"}
    sparsity = prefill_sparsity(path, data, chunks, L)

    line = {"metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config, "clocks": clocks,
            "e2e": {"value": replicas.whole_job_rate(world, L, ms_e2e) if ms_e2e else None, "unit": "tokens/s", "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "overlap": "two staging buffer sets, copies on a second stream",
                    "last_chunk_equals_resident_run": e2e_ok},
            "gpu_launches": args.steps * len(chunks) * path.launches_per_chunk,
            "roofline": roofline, "device_status": status,
            "selected_fraction_last_chunk": sel_frac, "sparse_prefill_flops": s6, "sparsity": sparsity,
            "kernel_ms_per_step": klass,
            "kernel_tflops": {"sparse_attn": fl_sparse / klass["sparse_attn"] / 1e9,
                              "local_attn": fl_local / klass["local_attn"] / 1e9},
            "indexer_scores_per_s": pairs * len(data.heads.ret_q_heads) / (klass["select"] * 1e-3)}

    if rank == 0 and not args.no_extras:
        # dense in-library baseline at the same shape
        step_dense()
        torch.cuda.synchronize()
        t_dense = min(ev_time_ms(step_dense, stream) for _ in range(2))
        line["dense_baseline"] = {"kernel": "attn_prefill_tc_kernel<dense> (tcgen05 + TMEM + TMA)",
                                  "ms_per_step": t_dense, "tokens_per_s": L / (t_dense * 1e-3),
                                  "tflops": fl_dense / t_dense / 1e9,
                                  "frac_of_bf16_peak": fl_dense / t_dense / 1e9 / peaks["bf16_tflops_sustained"],
                                  "peak": peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " (sustained bf16)",
                                  "speedup_sparse_vs_dense": t_dense / ms_per_step}
        # the paper's own prefill mode (Section 3.2): retrieval heads dense, local heads sink + window, index keys appended
        ret_kv = list(data.heads.ret_kv_heads)

        def step_paper():
            for (s, C) in chunks:
                rb.rtp_index_keys(path.ctx, path.params, path.cache, k_pre[s:s + C], data.w_k, path.tok_seq[:C],
                                  path.pos_all[s:s + C])
                rb.rtp_dense_attn_prefill(path.ctx, path.params, path.cache, data.q[s:s + C], 0, s, C, ret_kv,
                                          out[s:s + C], None, path.status)
                rb.rtp_local_attn(path.ctx, path.params, path.cache, data.q[s:s + C], None, None, 0, s, C, out[s:s + C],
                                  None, path.workspace, path.status)

        step_paper()
        torch.cuda.synchronize()
        t_paper = min(ev_time_ms(step_paper, stream) for _ in range(2))
        line["paper_prefill_mode"] = {"what": "retrieval heads dense + local heads sink/window + index-key append",
                                      "ms_per_step": t_paper, "tokens_per_s": L / (t_paper * 1e-3),
                                      "speedup_vs_dense": t_dense / t_paper}
        # the block-wise selection of Section 3.4 (whole pages instead of tokens) on the same workload
        def step_blocks():
            for (s, C) in chunks:
                path.run_chunk_blocks(s, C, data.q[s:s + C], k_pre[s:s + C], out[s:s + C])

        step_blocks()
        torch.cuda.synchronize()
        t_blocks = min(ev_time_ms(step_blocks, stream) for _ in range(2))
        kb = {"select_blocks": 0.0, "attn_blocks": 0.0}
        n_blk_sel = torch.zeros((), dtype=torch.float64, device=device)
        n_blk_all = 0.0
        for (s, C) in chunks:
            q = data.q[s:s + C]
            kb["select_blocks"] += ev_time_ms(lambda: rb.rtp_topp_select_blocks(path.ctx, path.params, path.cache, q, data.w_q, 0, s, C, path.blk_mask[:C], path.sel_cnt[:C], path.sel_mass[:C], path.sel_thr[:C], path.sel_tie[:C], path.status, path.blk_ws), stream)
            kb["attn_blocks"] += ev_time_ms(lambda: rb.rtp_sparse_attn_prefill_blocks(path.ctx, path.params, path.cache, q, 0, s, C, path.blk_mask[:C], out[s:s + C], None, path.status), stream)
            n_blk_sel += path.sel_cnt[:C].sum(dtype=torch.float64)
            n_blk_all += float(((torch.arange(s, s + C, device=device) // 64 + 1).sum() * len(data.heads.ret_q_heads)).item())
        line["block_topp_path"] = {"what": "index keys + block-wise top-p (one bit per row, head, page) + attention over the selected pages + local heads",
                                   "ms_per_step": t_blocks, "tokens_per_s": L / (t_blocks * 1e-3),
                                   "speedup_vs_dense": t_dense / t_blocks, "kernel_ms_per_step": kb,
                                   "selected_block_fraction": float(n_blk_sel.item()) / n_blk_all,
                                   "attn_tflops": fl_sparse / kb["attn_blocks"] / 1e9,
                                   "status": path.status_code()}
        if not c4:   # the 1M run stops at the comparators: no CPU sample, no decode points
            # CPU oracle on a bounded sample of the same workload
            rows = np.linspace(L // 8, L - 1, 160).astype(np.int64)
            v, done, secs, used = cpu_oracle_prefill(data, L, rows, budget_s=20.0)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": used, "cores_available": n_cores,
                                    "kind": "oracle (numpy, fp64)",
                                    "sample": f"{done} query rows x 32 heads spread over the sequence ({secs:.1f} s), "
                                              f"extrapolated per token"}
            del path, data, out, k_pre
            torch.cuda.empty_cache()
            dec = []
            dec.append(bench_decode_point(device, "c2_decode_batched_gqa", 32768, 8, 0.95, 0.1, 2048, True))
            dec.append(bench_decode_point(device, "c5_decode_b4_512k", 524288, 4, 0.9, 0.05, 4096, False))
            dec.append(bench_decode_point(device, "c1_sized_decode_b1_4k", 4096, 1, 0.9, 0.05, 2048, False, variants=False))
            line["decode"] = dec
    elif "cpu_baseline" not in line:
        line["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
