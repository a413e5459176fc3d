"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and lays tensors out in memory; it holds
none of the method's arithmetic (no scores, no softmax, no selection, no
attention).  Both the CUDA path and the CPU oracle are fed from here, so that
they see the same bit patterns.

Conventions
-----------
* bf16 tensors are numpy ``uint16`` arrays holding the raw bit patterns.
* "Logical" K/V of one sequence are ``[L, Hkv, 128]``; the paged cache is
  ``[num_pages, Hkv, 64, 128]`` (K and V separately) plus an index-key cache
  ``[num_pages, n_index_heads, 64, 16]`` that shares the block table.
* A *retrieval KV head* makes all its G query heads retrieval heads (or, with
  ``ret_per_group``, only the first few of them: a mixed group).  Each
  retrieval query head has its own ``W_q``; each index head (one per retrieval
  KV head) has one ``W_k``.  The generators tie ``W_q = W_k`` inside a group so
  that a planted key aligned with a query really gets a high projected score
  (Eq. 4 with independent random projections has zero-mean needle scores).
* Pre-RoPE and post-RoPE tensors coincide (``q_pre = q``, ``k_pre = K``): RoPE
  is outside the path.

The five ``config_*`` functions mirror the benchmark configurations: single
decode step with needles (1), batched GQA decode with peaked and flat queries
(2), chunked prefill with a rank-16 dominant key subspace (3), long prefill
with planted needles (4) and the long-context decode sweep (5).  Every one of
them takes the context length as an argument, so that the tests can run the
same recipe at sizes the CPU oracle finishes in seconds.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from statistics import NormalDist

import numpy as np

HEAD_DIM = 128
INDEX_DIM = 16
PAGE_SIZE = 64
BASE_SEED = 20260516


# --------------------------------------------------------------------------
# bf16 bit patterns (data preparation only)
# --------------------------------------------------------------------------
def to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (round to nearest even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def from_bf16(u: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------
@dataclass
class HeadMap:
    """Static head partition (an input of the method, fixed per model)."""
    n_q_heads: int
    n_kv_heads: int
    ret_kv_heads: list            # KV heads whose query heads are retrieval heads
    n_sink: int = 4
    window: int = 8192
    # > 0: a mixed group: only the first ret_per_group query heads of a retrieval KV head are retrieval heads, the
    # others of the group attend locally (the KV head is then also a local KV head)
    ret_per_group: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def _rpg(self) -> int:
        return self.ret_per_group if 0 < self.ret_per_group < self.group else self.group

    @property
    def local_kv_heads(self) -> list:
        mixed = self._rpg < self.group
        return [h for h in range(self.n_kv_heads) if mixed or h not in self.ret_kv_heads]

    @property
    def ret_q_heads(self) -> list:
        g = self.group
        return [kv * g + j for kv in self.ret_kv_heads for j in range(self._rpg)]

    @property
    def local_q_heads(self) -> list:
        ret = set(self.ret_q_heads)
        return [kv * self.group + j for kv in self.local_kv_heads for j in range(self.group) if kv * self.group + j not in ret]

    @property
    def n_index_heads(self) -> int:
        return len(self.ret_kv_heads)

    @property
    def q_head_to_index_head(self) -> list:
        """For retrieval query head number i (position in ret_q_heads)."""
        return [i // self._rpg for i in range(len(self.ret_q_heads))]

    @property
    def index_head_kv(self) -> list:
        return list(self.ret_kv_heads)


@dataclass
class Workload:
    name: str
    heads: HeadMap
    top_p: float
    score_scale: float
    sm_scale: float
    seq_lens: np.ndarray                 # int32 [B]
    k: list                              # per sequence: uint16 [L, Hkv, 128]
    v: list                              # per sequence: uint16 [L, Hkv, 128]
    w_q: np.ndarray                      # uint16 [n_ret_q, 128, 16]
    w_k: np.ndarray                      # uint16 [n_index_heads, 128, 16]
    q: np.ndarray                        # uint16 [R, Hq, 128] query rows
    row_seq: np.ndarray                  # int32 [R]
    row_pos: np.ndarray                  # int32 [R]  (row sees keys 0..row_pos)
    seed: int = 0
    notes: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.k)


@dataclass
class PagedCache:
    k_pages: np.ndarray                  # uint16 [num_pages, Hkv, 64, 128]
    v_pages: np.ndarray                  # uint16 [num_pages, Hkv, 64, 128]
    block_table: np.ndarray              # int32 [B, max_pages]
    seq_lens: np.ndarray                 # int32 [B]
    num_pages: int


def build_paged_cache(k: list, v: list, seed: int, capacity: list | None = None,
                      spare_pages: int = 1) -> PagedCache:
    """Scatter logical K/V into a paged cache through a random page permutation.

    ``capacity[b]`` (tokens) reserves pages beyond ``len(k[b])`` for appends.
    """
    B = len(k)
    hkv = k[0].shape[1]
    cap = [int(k[b].shape[0]) for b in range(B)] if capacity is None else [int(c) for c in capacity]
    n_pages_seq = [(c + PAGE_SIZE - 1) // PAGE_SIZE for c in cap]
    max_pages = max(1, max(n_pages_seq))
    num_pages = sum(n_pages_seq) + spare_pages
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x9E3779B9))
    perm = rng.permutation(num_pages).astype(np.int32)
    block_table = np.zeros((B, max_pages), dtype=np.int32)
    k_pages = np.zeros((num_pages, hkv, PAGE_SIZE, HEAD_DIM), dtype=np.uint16)
    v_pages = np.zeros((num_pages, hkv, PAGE_SIZE, HEAD_DIM), dtype=np.uint16)
    nxt = 0
    for b in range(B):
        L = int(k[b].shape[0])
        phys = perm[nxt: nxt + n_pages_seq[b]]
        nxt += n_pages_seq[b]
        block_table[b, : n_pages_seq[b]] = phys
        full = L // PAGE_SIZE
        if full:
            kk = k[b][: full * PAGE_SIZE].reshape(full, PAGE_SIZE, hkv, HEAD_DIM)
            vv = v[b][: full * PAGE_SIZE].reshape(full, PAGE_SIZE, hkv, HEAD_DIM)
            k_pages[phys[:full]] = np.transpose(kk, (0, 2, 1, 3))
            v_pages[phys[:full]] = np.transpose(vv, (0, 2, 1, 3))
        rem = L - full * PAGE_SIZE
        if rem:
            k_pages[phys[full], :, :rem, :] = np.transpose(k[b][full * PAGE_SIZE:], (1, 0, 2))
            v_pages[phys[full], :, :rem, :] = np.transpose(v[b][full * PAGE_SIZE:], (1, 0, 2))
    seq_lens = np.array([int(k[b].shape[0]) for b in range(B)], dtype=np.int32)
    return PagedCache(k_pages, v_pages, block_table, seq_lens, num_pages)


def gather_index_keys(ikey_pages: np.ndarray, block_table: np.ndarray, seq: int, L: int) -> np.ndarray:
    """Paged index-key cache -> logical ``[L, n_index_heads, 16]`` of one sequence."""
    n_pages = (L + PAGE_SIZE - 1) // PAGE_SIZE
    if n_pages == 0:
        return np.zeros((0, ikey_pages.shape[1], INDEX_DIM), dtype=np.uint16)
    phys = block_table[seq, :n_pages]
    x = ikey_pages[phys]                                   # [n_pages, nih, 64, 16]
    x = np.transpose(x, (0, 2, 1, 3)).reshape(n_pages * PAGE_SIZE, ikey_pages.shape[1], INDEX_DIM)
    return np.ascontiguousarray(x[:L])


# --------------------------------------------------------------------------
# random helpers
# --------------------------------------------------------------------------
def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _unit(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _normal(rng, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def _needle_key(rng, q_dir: np.ndarray, cos: float = 0.8) -> np.ndarray:
    """A key of norm sqrt(128) at cosine ``cos`` to the unit vector ``q_dir``."""
    g = _normal(rng, q_dir.shape)
    g = g - (g @ q_dir) * q_dir
    g = _unit(g)
    return np.sqrt(HEAD_DIM).astype(np.float32) * (cos * q_dir + np.sqrt(1.0 - cos * cos) * g)


def sigma_for_fraction(p: float, frac: float) -> float:
    """Score standard deviation at which iid Gaussian scores put the top-p cut
    at the given selected fraction (closed form for a lognormal mass profile)."""
    nd = NormalDist()
    return nd.inv_cdf(p) + nd.inv_cdf(1.0 - frac)


# --------------------------------------------------------------------------
# configuration 1: single decode step, one retrieval head, planted needles
# --------------------------------------------------------------------------
def config_1(L: int = 4096, n_needles: int = 8, seed: int = BASE_SEED + 1, top_p: float = 0.9) -> Workload:
    rng = _rng(seed)
    heads = HeadMap(n_q_heads=1, n_kv_heads=1, ret_kv_heads=[0], n_sink=4, window=8192)
    W = _normal(rng, (HEAD_DIM, INDEX_DIM)) / np.sqrt(np.float32(HEAD_DIM))
    a = _normal(rng, (INDEX_DIM,))
    q_dir = _unit(W @ a)
    q = np.sqrt(np.float32(HEAD_DIM)) * q_dir
    K = _normal(rng, (L, 1, HEAD_DIM))
    V = _normal(rng, (L, 1, HEAD_DIM))
    pos = rng.choice(L, size=min(n_needles, L), replace=False)
    for n in pos:
        K[n, 0] = _needle_key(rng, q_dir)
    wl = Workload(
        name="c1_decode_single", heads=heads, top_p=top_p, score_scale=0.125,
        sm_scale=1.0 / np.sqrt(HEAD_DIM), seq_lens=np.array([L], np.int32),
        k=[to_bf16(K)], v=[to_bf16(V)],
        w_q=to_bf16(W)[None], w_k=to_bf16(W)[None],
        q=to_bf16(q)[None, None], row_seq=np.array([0], np.int32), row_pos=np.array([L - 1], np.int32),
        seed=seed, notes={"needles": np.sort(pos)})
    return wl


# --------------------------------------------------------------------------
# configuration 2: batched GQA decode, half peaked / half flat
# --------------------------------------------------------------------------
def config_2(L: int = 32768, batch: int = 8, n_q_heads: int = 32, n_kv_heads: int = 8,
             ret_kv_heads=(0, 1), window: int = 2048, top_p: float = 0.95,
             flat_sigma: float = 2.5, seed: int = BASE_SEED + 2,
             needle_range=(16, 64), ret_per_group: int = 0) -> Workload:
    rng = _rng(seed)
    heads = HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), n_sink=4, window=window, ret_per_group=ret_per_group)
    g = heads.group
    scale = 0.125
    W = [_normal(rng, (HEAD_DIM, INDEX_DIM)) / np.sqrt(np.float32(HEAD_DIM)) for _ in heads.ret_kv_heads]
    q = _normal(rng, (batch, n_q_heads, HEAD_DIM))
    ks, vs = [], []
    needles = {}
    for b in range(batch):
        K = _normal(rng, (L, n_kv_heads, HEAD_DIM))
        V = _normal(rng, (L, n_kv_heads, HEAD_DIM))
        peaked = b < batch // 2
        for ih, kv in enumerate(heads.ret_kv_heads):
            free = rng.permutation(L)
            used = 0
            for j in range(g):
                h = kv * g + j
                a = _normal(rng, (INDEX_DIM,))
                q_dir = _unit(W[ih] @ a)
                if peaked:
                    q[b, h] = np.sqrt(np.float32(HEAD_DIM)) * q_dir
                    n_n = int(rng.integers(needle_range[0], needle_range[1] + 1))
                    n_n = min(n_n, max(1, L // (4 * g)))
                    pos = free[used: used + n_n]; used += n_n
                    for n in pos:
                        K[n, kv] = _needle_key(rng, q_dir)
                    needles[(b, h)] = np.sort(pos)
                else:
                    # flat: projected score std = scale * |W^T q| = flat_sigma
                    qt_norm = np.linalg.norm(W[ih].T @ q_dir)
                    q[b, h] = (flat_sigma / (scale * qt_norm)) * q_dir
        ks.append(to_bf16(K)); vs.append(to_bf16(V))
    w_k = to_bf16(np.stack(W))
    w_q = to_bf16(np.stack([W[i] for i in heads.q_head_to_index_head]))
    return Workload(
        name="c2_decode_batched_gqa", heads=heads, top_p=top_p, score_scale=scale,
        sm_scale=1.0 / np.sqrt(HEAD_DIM), seq_lens=np.full(batch, L, np.int32),
        k=ks, v=vs, w_q=w_q, w_k=w_k, q=to_bf16(q),
        row_seq=np.arange(batch, dtype=np.int32), row_pos=np.full(batch, L - 1, np.int32),
        seed=seed, notes={"needles": needles})


# --------------------------------------------------------------------------
# configuration 3: chunked prefill, rank-16 dominant key subspace
# --------------------------------------------------------------------------
def config_3(L: int = 131072, n_q_heads: int = 32, n_kv_heads: int = 8, ret_kv_heads=(0, 1),
             window: int = 8192, top_p: float = 0.9, score_scale: float = 0.146,
             seed: int = BASE_SEED + 3, ret_per_group: int = 0) -> Workload:
    rng = _rng(seed)
    heads = HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), n_sink=4, window=window, ret_per_group=ret_per_group)
    U = []
    for _ in range(n_kv_heads):
        a, _r = np.linalg.qr(rng.standard_normal((HEAD_DIM, INDEX_DIM)))
        U.append(a.astype(np.float32))
    g = heads.group
    K = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    Q = _normal(rng, (L, n_q_heads, HEAD_DIM))
    for kv in range(n_kv_heads):
        z = _normal(rng, (L, INDEX_DIM))
        K[:, kv] += 2.0 * (z @ U[kv].T)
        for j in range(g):
            zq = _normal(rng, (L, INDEX_DIM))
            Q[:, kv * g + j] += 2.0 * (zq @ U[kv].T)
    V = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    w_k = to_bf16(np.stack([U[kv] for kv in heads.ret_kv_heads]))
    w_q = to_bf16(np.stack([U[heads.ret_kv_heads[i]] for i in heads.q_head_to_index_head]))
    return Workload(
        name="c3_prefill_chunked", heads=heads, top_p=top_p, score_scale=score_scale,
        sm_scale=1.0 / np.sqrt(HEAD_DIM), seq_lens=np.array([L], np.int32),
        k=[to_bf16(K)], v=[to_bf16(V)], w_q=w_q, w_k=w_k, q=to_bf16(Q),
        row_seq=np.zeros(L, np.int32), row_pos=np.arange(L, dtype=np.int32), seed=seed)


def config_grid_ties(L: int = 3000, n_q_heads: int = 32, n_kv_heads: int = 8, ret_kv_heads=(0, 1), window: int = 512,
                     top_p: float = 0.9, amp: int = 3, seed: int = BASE_SEED + 33) -> Workload:
    """A stress input for equal and grid-aligned scores (not one of the paper's workloads): the indexer's matrices pick
    the first 16 coordinates, and those coordinates of the retrieval heads' keys and queries are small integers, so with
    the temperature 1/8 every score is a multiple of 1/8, half of them lie exactly between two quarter-wide score bins,
    and every value is shared by many keys.  The other coordinates, the values and the local heads are N(0,1)."""
    rng = _rng(seed)
    heads = HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), n_sink=4, window=window)
    g = heads.group
    K = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    V = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    Q = _normal(rng, (L, n_q_heads, HEAD_DIM))
    for kv in heads.ret_kv_heads:
        K[:, kv, :INDEX_DIM] = rng.integers(-amp, amp + 1, size=(L, INDEX_DIM)).astype(np.float32)
        for j in range(g):
            Q[:, kv * g + j, :INDEX_DIM] = rng.integers(-amp, amp + 1, size=(L, INDEX_DIM)).astype(np.float32)
    sel = np.zeros((HEAD_DIM, INDEX_DIM), np.float32)
    sel[np.arange(INDEX_DIM), np.arange(INDEX_DIM)] = 1.0
    w_k = to_bf16(np.stack([sel for _ in heads.ret_kv_heads]))
    w_q = to_bf16(np.stack([sel for _ in heads.q_head_to_index_head]))
    return Workload(
        name="grid_ties", heads=heads, top_p=top_p, score_scale=0.125, sm_scale=1.0 / np.sqrt(HEAD_DIM),
        seq_lens=np.array([L], np.int32), k=[to_bf16(K)], v=[to_bf16(V)], w_q=w_q, w_k=w_k, q=to_bf16(Q),
        row_seq=np.zeros(L, np.int32), row_pos=np.arange(L, dtype=np.int32), seed=seed)


# --------------------------------------------------------------------------
# configuration 4: long prefill with planted needles matched to query rows
# --------------------------------------------------------------------------
def config_4(L: int = 1048576, n_needles: int = 1024, n_q_heads: int = 32, n_kv_heads: int = 8,
             ret_kv_heads=(0,), window: int = 8192, top_p: float = 0.9,
             flat_sigma: float = 3.0, seed: int = BASE_SEED + 4) -> Workload:
    rng = _rng(seed)
    heads = HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), n_sink=4, window=window)
    g = heads.group
    scale = 0.125
    W = [_normal(rng, (HEAD_DIM, INDEX_DIM)) / np.sqrt(np.float32(HEAD_DIM)) for _ in heads.ret_kv_heads]
    K = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    V = _normal(rng, (L, n_kv_heads, HEAD_DIM))
    Q = _normal(rng, (L, n_q_heads, HEAD_DIM))
    # flat rows of retrieval heads: projected-score std = flat_sigma
    for ih, kv in enumerate(heads.ret_kv_heads):
        for j in range(g):
            h = kv * g + j
            a = _normal(rng, (L, INDEX_DIM))
            d = _unit(a @ W[ih].T)
            qt = np.linalg.norm(d @ W[ih], axis=-1, keepdims=True)
            Q[:, h] = (flat_sigma / (scale * qt)) * d
    n_needles = min(n_needles, max(1, L // 8))
    kpos = np.sort(rng.choice(L - 1, size=n_needles, replace=False))
    qrow = np.empty(n_needles, dtype=np.int64)
    taken = set()
    for i, n in enumerate(kpos):
        while True:
            r = int(rng.integers(n + 1, L))
            if r not in taken:
                taken.add(r); break
        qrow[i] = r
    for ih, kv in enumerate(heads.ret_kv_heads):
        for i, n in enumerate(kpos):
            a = _normal(rng, (INDEX_DIM,))
            q_dir = _unit(W[ih] @ a)
            K[n, kv] = _needle_key(rng, q_dir)
            for j in range(g):
                Q[qrow[i], kv * g + j] = np.sqrt(np.float32(HEAD_DIM)) * q_dir
    w_k = to_bf16(np.stack(W))
    w_q = to_bf16(np.stack([W[i] for i in heads.q_head_to_index_head]))
    return Workload(
        name="c4_prefill_long", heads=heads, top_p=top_p, score_scale=scale,
        sm_scale=1.0 / np.sqrt(HEAD_DIM), seq_lens=np.array([L], np.int32),
        k=[to_bf16(K)], v=[to_bf16(V)], w_q=w_q, w_k=w_k, q=to_bf16(Q),
        row_seq=np.zeros(L, np.int32), row_pos=np.arange(L, dtype=np.int32), seed=seed,
        notes={"needle_key_pos": kpos, "needle_query_row": qrow})


# --------------------------------------------------------------------------
# configuration 5: long-context decode sweep point
# --------------------------------------------------------------------------
def config_5(L: int = 131072, batch: int = 1, top_p: float = 0.9, frac: float = 0.05,
             n_q_heads: int = 32, n_kv_heads: int = 8, ret_kv_heads=(0, 1), window: int = 4096,
             seed: int = BASE_SEED + 5) -> Workload:
    """iid keys; the score temperature is set from the Gaussian closed form so
    that top-p keeps about ``frac`` of the context."""
    rng = _rng(seed)
    heads = HeadMap(n_q_heads, n_kv_heads, list(ret_kv_heads), n_sink=4, window=window)
    g = heads.group
    scale = 0.125
    sigma = sigma_for_fraction(top_p, frac)
    W = [_normal(rng, (HEAD_DIM, INDEX_DIM)) / np.sqrt(np.float32(HEAD_DIM)) for _ in heads.ret_kv_heads]
    q = _normal(rng, (batch, n_q_heads, HEAD_DIM))
    for b in range(batch):
        for ih, kv in enumerate(heads.ret_kv_heads):
            for j in range(g):
                a = _normal(rng, (INDEX_DIM,))
                d = _unit(W[ih] @ a)
                qt = np.linalg.norm(W[ih].T @ d)
                q[b, kv * g + j] = (sigma / (scale * qt)) * d
    ks = [to_bf16(_normal(rng, (L, n_kv_heads, HEAD_DIM))) for _ in range(batch)]
    vs = [to_bf16(_normal(rng, (L, n_kv_heads, HEAD_DIM))) for _ in range(batch)]
    w_k = to_bf16(np.stack(W))
    w_q = to_bf16(np.stack([W[i] for i in heads.q_head_to_index_head]))
    return Workload(
        name="c5_decode_sweep", heads=heads, top_p=top_p, score_scale=scale,
        sm_scale=1.0 / np.sqrt(HEAD_DIM), seq_lens=np.full(batch, L, np.int32),
        k=ks, v=vs, w_q=w_q, w_k=w_k, q=to_bf16(q),
        row_seq=np.arange(batch, dtype=np.int32), row_pos=np.full(batch, L - 1, np.int32),
        seed=seed, notes={"sigma": sigma, "target_fraction": frac})


def k_pre_for_index_heads(wl: Workload, seq: int, lo: int = 0, hi: int | None = None) -> np.ndarray:
    """Pre-RoPE keys of the index heads of one sequence: ``[hi-lo, n_index_heads, 128]``.

    The synthetic workloads apply no RoPE, so these are the cached keys of the
    retrieval KV heads."""
    hi = int(wl.k[seq].shape[0]) if hi is None else hi
    return np.ascontiguousarray(wl.k[seq][lo:hi][:, wl.heads.index_head_kv, :])
