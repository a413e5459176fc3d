"""Full-size synthetic workloads generated directly in device memory (torch used as an allocator
and random-number source only).  Same recipes as ``synth`` (which draws on the host with numpy and
is used at sizes the CPU oracle finishes in seconds); no method arithmetic here either.

The tensors are laid out exactly as the library wants them: paged K/V
``[num_pages, Hkv, 64, 128]`` behind a seeded random block table, queries ``[L, Hq, 128]``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

from . import synth

PAGE = synth.PAGE_SIZE


@dataclass
class DeviceData:
    name: str
    heads: synth.HeadMap
    top_p: float
    score_scale: float
    sm_scale: float
    seq_lens: torch.Tensor          # int32 [B]
    block_table: torch.Tensor       # int32 [B, max_pages]
    k_pages: torch.Tensor           # bf16 [num_pages, Hkv, 64, 128]
    v_pages: torch.Tensor
    w_q: torch.Tensor               # bf16 [n_ret, 128, 16]
    w_k: torch.Tensor               # bf16 [n_index_heads, 128, 16]
    q: torch.Tensor                 # bf16 [R, Hq, 128]
    row_seq: torch.Tensor           # int32 [R]
    row_pos: torch.Tensor           # int32 [R]
    seed: int
    notes: dict = field(default_factory=dict)

    @property
    def num_pages(self) -> int:
        return int(self.k_pages.shape[0])

    def logical_kv(self, seq: int, kv_head: int, lo: int = 0, hi: int | None = None):
        """K and V of one KV head of one sequence as host uint16 arrays [hi-lo, 128]."""
        L = int(self.seq_lens[seq])
        hi = L if hi is None else hi
        p0, p1 = lo // PAGE, (hi + PAGE - 1) // PAGE
        phys = self.block_table[seq, p0:p1].long()
        k = self.k_pages[phys, kv_head].reshape(-1, 128)[lo - p0 * PAGE: hi - p0 * PAGE]
        v = self.v_pages[phys, kv_head].reshape(-1, 128)[lo - p0 * PAGE: hi - p0 * PAGE]
        to_np = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        return to_np(k), to_np(v)

    def k_pre_rows(self, seq: int, lo: int, hi: int) -> torch.Tensor:
        """Pre-RoPE keys of the index heads for tokens lo..hi-1: bf16 [hi-lo, n_index_heads, 128]
        (the synthetic workloads apply no RoPE, so these are the cached keys of the retrieval KV heads)."""
        p0, p1 = lo // PAGE, (hi + PAGE - 1) // PAGE
        phys = self.block_table[seq, p0:p1].long()
        x = self.k_pages[phys][:, self.heads.index_head_kv]          # [pages, nih, 64, 128]
        x = x.permute(0, 2, 1, 3).reshape(-1, len(self.heads.index_head_kv), 128)
        return x[lo - p0 * PAGE: hi - p0 * PAGE].contiguous()


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _paged(B: int, L: int, n_kv: int, device, g):
    n_pages_seq = (L + PAGE - 1) // PAGE
    num_pages = B * n_pages_seq + 1
    perm = torch.randperm(num_pages, device=device, generator=g)[: B * n_pages_seq]
    block_table = perm.to(torch.int32).reshape(B, n_pages_seq).contiguous()
    return num_pages, block_table


def _fill_pages(pages: torch.Tensor, block_table: torch.Tensor, g, extra=None, chunk_pages: int = 2048):
    """pages[phys] = N(0,1) (+ extra(seq, logical page range) if given), bf16, a slab at a time."""
    B, nps = block_table.shape
    hkv = pages.shape[1]
    for b in range(B):
        for p0 in range(0, nps, chunk_pages):
            p1 = min(nps, p0 + chunk_pages)
            x = torch.randn((p1 - p0, hkv, PAGE, 128), device=pages.device, generator=g, dtype=torch.float32)
            if extra is not None:
                x = extra(b, p0, p1, x)
            pages[block_table[b, p0:p1].long()] = x.to(torch.bfloat16)


def config_3_device(L: int = 131072, device="cuda:0", seed: int = synth.BASE_SEED + 3, top_p: float = 0.9,
                    score_scale: float = 0.155, window: int = 8192, n_q_heads: int = 32, n_kv_heads: int = 8,
                    ret_kv_heads=(0, 1)) -> DeviceData:
    """Chunked-prefill workload: keys and queries have a rank-16 dominant subspace (4x variance)
    per KV head plus unit noise; the indexer projections are that subspace's orthonormal basis."""
    g = _gen(device, seed)
    heads = synth.HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), 4, window)
    grp = heads.group
    U = torch.stack([torch.linalg.qr(torch.randn((128, 16), device=device, generator=g))[0] for _ in range(n_kv_heads)])
    num_pages, bt = _paged(1, L, n_kv_heads, device, g)
    k_pages = torch.empty((num_pages, n_kv_heads, PAGE, 128), device=device, dtype=torch.bfloat16)
    v_pages = torch.empty_like(k_pages)

    def low_rank(b, p0, p1, x):
        z = torch.randn((p1 - p0, n_kv_heads, PAGE, 16), device=device, generator=g)
        return x + 2.0 * torch.einsum("phtr,hdr->phtd", z, U)

    _fill_pages(k_pages, bt, g, low_rank)
    _fill_pages(v_pages, bt, g)
    q = torch.empty((L, n_q_heads, 128), device=device, dtype=torch.bfloat16)
    for lo in range(0, L, 16384):
        hi = min(L, lo + 16384)
        x = torch.randn((hi - lo, n_q_heads, 128), device=device, generator=g)
        z = torch.randn((hi - lo, n_q_heads, 16), device=device, generator=g)
        Uq = U.repeat_interleave(grp, dim=0)                           # [Hq, 128, 16]
        q[lo:hi] = (x + 2.0 * torch.einsum("thr,hdr->thd", z, Uq)).to(torch.bfloat16)
    w_k = U[list(ret_kv_heads)].to(torch.bfloat16).contiguous()
    w_q = U[[heads.ret_kv_heads[i] for i in heads.q_head_to_index_head]].to(torch.bfloat16).contiguous()
    return DeviceData("c3_prefill_chunked", heads, top_p, score_scale, 1.0 / math.sqrt(128),
                      torch.tensor([L], dtype=torch.int32, device=device), bt, k_pages, v_pages, w_q, w_k, q,
                      torch.zeros(L, dtype=torch.int32, device=device),
                      torch.arange(L, dtype=torch.int32, device=device), seed)


def config_4_device(L: int = 1048576, device="cuda:0", seed: int = synth.BASE_SEED + 4, top_p: float = 0.9,
                    flat_sigma: float = 3.0, n_needles: int = 1024, window: int = 8192, n_q_heads: int = 32,
                    n_kv_heads: int = 8, ret_kv_heads=(0,), needle_gain: float = 2.0) -> DeviceData:
    """Long-prefill workload: N(0,1) keys, values and queries; on the retrieval KV heads every query head's rows are
    "flat" (a direction inside the indexer's subspace scaled so that the projected scores have standard deviation
    ``flat_sigma``), except for ``n_needles`` rows: a needle key (cosine 0.8 with a direction of the subspace) is
    planted at a uniformly drawn position and matched to a distinct later query row, whose four query heads of the
    group all point in the needle's direction (the same recipe as ``synth.config_4``, drawn on the device).  The matched
    rows' queries are ``needle_gain`` times as long as in the host recipe: with a million keys behind it a needle has to
    score about ln(1e6) higher than at a few thousand to carry most of its row's mass."""
    g = _gen(device, seed)
    heads = synth.HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), 4, window)
    grp = heads.group
    scale = 0.125
    W = torch.randn((len(ret_kv_heads), 128, 16), device=device, generator=g) / math.sqrt(128)
    num_pages, bt = _paged(1, L, n_kv_heads, device, g)
    k_pages = torch.empty((num_pages, n_kv_heads, PAGE, 128), device=device, dtype=torch.bfloat16)
    v_pages = torch.empty_like(k_pages)
    _fill_pages(k_pages, bt, g)
    _fill_pages(v_pages, bt, g)
    q = torch.empty((L, n_q_heads, 128), device=device, dtype=torch.bfloat16)
    ret_q = set(heads.ret_q_heads)
    for lo in range(0, L, 16384):
        hi = min(L, lo + 16384)
        x = torch.randn((hi - lo, n_q_heads, 128), device=device, generator=g)
        for ih, kv in enumerate(heads.ret_kv_heads):
            for j in range(grp):
                a = torch.randn((hi - lo, 16), device=device, generator=g)
                dvec = a @ W[ih].T
                dvec = dvec / dvec.norm(dim=-1, keepdim=True)
                qt = (dvec @ W[ih]).norm(dim=-1, keepdim=True)
                x[:, kv * grp + j] = flat_sigma / (scale * qt) * dvec
        q[lo:hi] = x.to(torch.bfloat16)
    # needles: key positions uniform without replacement, each matched to a distinct later query row
    cpu = np.random.Generator(np.random.PCG64(seed))
    n_needles = min(n_needles, max(1, L // 8))
    kpos = np.sort(cpu.choice(L - 1, size=n_needles, replace=False))
    qrow = np.empty(n_needles, dtype=np.int64)
    taken = set()
    for i, n in enumerate(kpos):
        while True:
            r = int(cpu.integers(n + 1, L))
            if r not in taken:
                taken.add(r)
                break
        qrow[i] = r
    kpos_t = torch.from_numpy(kpos).to(device)
    qrow_t = torch.from_numpy(qrow).to(device)
    for ih, kv in enumerate(heads.ret_kv_heads):
        a = torch.randn((n_needles, 16), device=device, generator=g)
        q_dir = a @ W[ih].T
        q_dir = q_dir / q_dir.norm(dim=-1, keepdim=True)
        gg = torch.randn((n_needles, 128), device=device, generator=g)
        gg = gg - (gg * q_dir).sum(-1, keepdim=True) * q_dir
        gg = gg / gg.norm(dim=-1, keepdim=True)
        needle = math.sqrt(128.0) * (0.8 * q_dir + 0.6 * gg)
        phys = bt[0, (kpos_t // PAGE)].long()
        k_pages[phys, kv, (kpos_t % PAGE)] = needle.to(torch.bfloat16)
        for j in range(grp):
            q[qrow_t, kv * grp + j] = (needle_gain * math.sqrt(128.0) * q_dir).to(torch.bfloat16)
    w_k = W.to(torch.bfloat16).contiguous()
    w_q = W[[heads.q_head_to_index_head[i] for i in range(len(heads.ret_q_heads))]].to(torch.bfloat16).contiguous()
    return DeviceData("c4_prefill_long", heads, top_p, scale, 1.0 / math.sqrt(128),
                      torch.tensor([L], dtype=torch.int32, device=device), bt, k_pages, v_pages, w_q, w_k, q,
                      torch.zeros(L, dtype=torch.int32, device=device),
                      torch.arange(L, dtype=torch.int32, device=device), seed,
                      {"needle_key_pos": kpos, "needle_query_row": qrow, "flat_sigma": flat_sigma, "needle_gain": needle_gain})


def decode_device(L: int, batch: int, top_p: float, frac: float, window: int, device="cuda:0",
                  seed: int = synth.BASE_SEED + 5, n_q_heads: int = 32, n_kv_heads: int = 8,
                  ret_kv_heads=(0, 1), peaked_half: bool = False, name: str = "c5_decode_sweep") -> DeviceData:
    """Decode workloads (batched GQA decode and the long-context sweep): iid keys; the projected-score
    temperature is set from the Gaussian closed form so that top-p keeps about ``frac`` of the context.
    With ``peaked_half`` the first half of the batch instead gets 16..64 planted keys per retrieval head."""
    g = _gen(device, seed)
    heads = synth.HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), 4, window)
    grp = heads.group
    scale = 0.125
    sigma = synth.sigma_for_fraction(top_p, frac)
    W = torch.randn((len(ret_kv_heads), 128, 16), device=device, generator=g) / math.sqrt(128)
    num_pages, bt = _paged(batch, L, n_kv_heads, device, g)
    k_pages = torch.empty((num_pages, n_kv_heads, PAGE, 128), device=device, dtype=torch.bfloat16)
    v_pages = torch.empty_like(k_pages)
    _fill_pages(k_pages, bt, g)
    _fill_pages(v_pages, bt, g)
    q = torch.randn((batch, n_q_heads, 128), device=device, generator=g)
    cpu = np.random.Generator(np.random.PCG64(seed))
    dirs, qt_norms = [], []
    for i, h in enumerate(heads.ret_q_heads):
        ih = i // grp
        a = torch.randn((batch, 16), device=device, generator=g)
        dvec = a @ W[ih].T
        dvec = dvec / dvec.norm(dim=-1, keepdim=True)
        qt = (dvec @ W[ih]).norm(dim=-1, keepdim=True)
        q[:, h] = sigma / (scale * qt) * dvec
        dirs.append(dvec)
        qt_norms.append(qt)
        if peaked_half:
            for b in range(batch // 2):
                q[b, h] = math.sqrt(128.0) * dvec[b]
                n_n = int(cpu.integers(16, 65))
                pos = torch.from_numpy(cpu.choice(L, size=n_n, replace=False)).to(device)
                gg = torch.randn((n_n, 128), device=device, generator=g)
                gg = gg - (gg @ dvec[b])[:, None] * dvec[b][None, :]
                gg = gg / gg.norm(dim=-1, keepdim=True)
                needle = math.sqrt(128.0) * (0.8 * dvec[b][None, :] + 0.6 * gg)
                phys = bt[b, (pos // PAGE)].long()
                k_pages[phys, heads.ret_kv_heads[ih], (pos % PAGE)] = needle.to(torch.bfloat16)
    w_k = W.to(torch.bfloat16).contiguous()
    w_q = W[[i // grp for i in range(len(heads.ret_q_heads))]].to(torch.bfloat16).contiguous()
    return DeviceData(name, heads, top_p, scale, 1.0 / math.sqrt(128),
                      torch.full((batch,), L, dtype=torch.int32, device=device), bt, k_pages, v_pages, w_q, w_k,
                      q.to(torch.bfloat16), torch.arange(batch, dtype=torch.int32, device=device),
                      torch.full((batch,), L - 1, dtype=torch.int32, device=device), seed,
                      {"sigma": sigma, "target_fraction": frac, "ret_dirs": dirs, "ret_qt_norms": qt_norms})


def decode_retarget(data: DeviceData, top_p: float, frac: float) -> DeviceData:
    """The same cache and query directions as ``data`` (a ``decode_device`` workload without planted keys) at another
    top-p and another score temperature: only the lengths of the retrieval heads' queries change."""
    import dataclasses
    sigma = synth.sigma_for_fraction(top_p, frac)
    q = data.q.clone()
    for i, h in enumerate(data.heads.ret_q_heads):
        q[:, h] = (sigma / (data.score_scale * data.notes["ret_qt_norms"][i]) * data.notes["ret_dirs"][i]).to(q.dtype)
    notes = dict(data.notes, sigma=sigma, target_fraction=frac)
    return dataclasses.replace(data, top_p=top_p, q=q, notes=notes)
