"""CPU oracle for the sparse-attention hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the path computes, written from
the paper's definitions.  It shares no code with the CUDA library and must
never be imported by the product path; only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it.

What it follows
---------------
* ``index_project``      Eq. 4, the low-rank projection  W^K k_pre  /  W^Q q_pre
                         (Section 3.2), stored in bf16 as the index-key cache is.
* ``index_scores``       Eq. 4, s_h(m, n) = (W^Q q_pre)^T (W^K k_pre), times an
                         optional temperature (1.0 in the paper).
* ``softmax_mass``       the probability distribution that the projected scores
                         define and that stage-1 training fits to the full
                         attention distribution (Section 3.3): a plain softmax
                         of s_h(m, .) over the causal keys.
* ``topp_select``        Eq. 5, S_h(m) = Top-P(s_h(m, .), p): the shortest prefix
                         of the keys, taken in order of decreasing score, whose
                         softmax mass reaches p.  Token level (Section 3 speaks
                         of token-level sparse computation; the 64-token blocks
                         of Section 3.4 are a kernel approximation).
* ``block_lse`` / ``topp_select_blocks``
                         Section 3.4, the block-wise form of Eq. 5: the keys are
                         cut into blocks of 64, every block is reduced to a
                         log-sum-exp pair (m_b, l_b), blocks are taken in order
                         of decreasing m_b until their softmax mass reaches p.
* ``topk_select``        Section 4.1, the fixed-budget variant the paper compares
                         with ("w/ top-k", k = 4096): the k largest scores.
* ``forced_tokens`` / ``with_forced``
                         an optional variant that is not in Eq. 5: the first
                         n_sink and the newest n_recent keys joined to a
                         selected set (off by default: the paper forces nothing).
* ``e4m3_encode`` / ``e4m3_decode`` / ``index_project_e4m3`` / ``index_scores_e4m3``
                         an option that is not in the paper: the index-key cache
                         held as 8-bit floats (E4M3), Eq. 4 evaluated on the
                         decoded keys.
* ``attention_over_set`` Eq. 5, softmax(q.k/sqrt(d_h)) restricted to S, times V.
* ``local_set``          Section 3.2 / Table 2: attention sinks plus a sliding
                         window on local heads.
* ``dense_set``          ordinary causal attention (what retrieval heads do in
                         the paper's prefill; the in-library comparator).

Readings taken where the paper is silent (each also listed in the design notes):
no extra scale inside the top-p softmax; ties broken towards the smaller token
index; p = 1 keeps every causal key; the selection is never empty; sinks, the
recent window and the query's own position are NOT forced into a retrieval
head's set; the block-wise selection orders blocks by their maximum score m_b
(the quantity the kernel of Section 3.4 indexes its histogram by), exactly
rather than through 256 bins, with ties towards the smaller block index, and
a block's mass is l_b exp(m_b - M) / Z; a query at position m sees keys 0..m; the window is the last W
positions including m; query head h reads KV head h // G.

Pins (tests/test_oracle_*.py): brute force over all subsets for tiny L, closed
forms (equal scores, geometric scores, one dominant score, Gaussian scores),
shift / permutation / monotonicity invariants, dense attention against
torch's scaled_dot_product_attention, boolean-mask SDPA for the local pattern,
the matrix-product identity for the indexer; for the block-wise selection:
equal blocks, one dominant block, block size 1 against the token-level rule,
brute force over all block subsets in m_b order; for the fixed-budget selector:
numpy's argpartition on distinct scores, the count rule, the tie rule on equal
scores, agreement with Top-P at the p that its own mass defines; for the forced
positions: their number in closed form and the subset / union laws; for the 8-bit
keys: all codes and a dense sample of reals against torch's float8_e4m3fn
conversion, round trip of every finite code, ties, saturation, monotonicity.  The selection statistics the
paper prints (its Tables 1, 6, 7) depend on model activations that are not
available: parity unpinned for those numbers; they only shape synthetic data.

All floating point is fp64 except where the method fixes a storage type:
projected keys/queries are rounded to bf16, scores are rounded once to fp32.
"""
from __future__ import annotations

import numpy as np

HEAD_DIM = 128
INDEX_DIM = 16


# ---------------------------------------------------------------- bf16 <-> float
def bf16_to_f64(u: np.ndarray) -> np.ndarray:
    u32 = np.asarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit pattern (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


# ---------------------------------------------------------------- Eq. 4: indexer
def index_project(x_bf16: np.ndarray, w_bf16: np.ndarray) -> np.ndarray:
    """Low-rank projection of pre-RoPE features (Eq. 4).

    x_bf16: [..., 128] bf16 bits; w_bf16: [128, 16] bf16 bits (the paper's
    W in R^{r x d_h}, stored transposed).  Returns [..., 16] bf16 bits:
    the sum is taken in fp64, rounded to fp32 and then to bf16.
    """
    x = bf16_to_f64(x_bf16)
    w = bf16_to_f64(w_bf16)
    y = x @ w
    return f32_to_bf16(y.astype(np.float32))


def index_scores(qt_bf16: np.ndarray, kt_bf16: np.ndarray, score_scale: float = 1.0) -> np.ndarray:
    """s(m, n) for one query row against keys 0..n-1 (Eq. 4).

    qt_bf16: [16]; kt_bf16: [n, 16].  Returns float32 [n]: the 16-term sum and
    the temperature are applied in fp64 and the result is rounded once.
    """
    q = bf16_to_f64(qt_bf16)
    k = bf16_to_f64(kt_bf16)
    return (float(score_scale) * (k @ q)).astype(np.float32)


# ---------------------------------------------------------------- 8-bit index keys (an option, not in the paper)
# The index-key cache may hold the projected keys as 8-bit floats, 16 bytes per token and index head: the format is
# E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; codes 0x7f / 0xff are NaN; largest
# finite magnitude 448; subnormals m / 8 * 2^-6).
def e4m3_decode(c: np.ndarray) -> np.ndarray:
    """E4M3 codes (uint8) -> float64, exactly."""
    c = np.asarray(c, dtype=np.uint8).astype(np.int64)
    e, m = (c >> 3) & 15, c & 7
    mag = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((c & 0x7F) == 0x7F, np.nan, mag)
    return np.where((c >> 7) == 1, -mag, mag)


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Finite reals -> E4M3 codes: the nearest representable value, a tie going to the code with an even mantissa,
    magnitudes beyond 448 saturating at 448; the sign bit is the sign of x (so a small negative number gives -0)."""
    x = np.asarray(x, dtype=np.float64)
    grid = e4m3_decode(np.arange(0, 127, dtype=np.uint8))          # the 127 finite non-negative values, ascending
    a = np.minimum(np.abs(x), 448.0)
    hi = np.clip(np.searchsorted(grid, a, side="left"), 1, 126)     # grid[hi-1] <= a <= grid[hi] (or a == grid[0])
    lo = hi - 1
    d_lo, d_hi = a - grid[lo], grid[hi] - a
    code = np.where(d_lo < d_hi, lo, np.where(d_hi < d_lo, hi, np.where(lo % 2 == 0, lo, hi)))
    return (code | np.where(np.signbit(x), 0x80, 0)).astype(np.uint8)


def index_project_e4m3(x_bf16: np.ndarray, w_bf16: np.ndarray) -> np.ndarray:
    """The projection of ``index_project`` stored as E4M3 codes: the fp64 sum is rounded to fp32, then encoded."""
    y = (bf16_to_f64(x_bf16) @ bf16_to_f64(w_bf16)).astype(np.float32)
    return e4m3_encode(y)


def index_scores_e4m3(qt_bf16: np.ndarray, k8: np.ndarray, score_scale: float = 1.0) -> np.ndarray:
    """Scores of one query row against 8-bit index keys: the bf16 projected query is taken in fp16 (exact for
    magnitudes in [2^-14, 65504], which is every value a projection produces in practice; smaller ones round to
    multiples of 2^-24), the keys are decoded exactly; the 16-term sum and the temperature are applied in fp64 and
    the result is rounded once, as for bf16 keys."""
    q = bf16_to_f64(qt_bf16).astype(np.float16).astype(np.float64)
    k = e4m3_decode(k8)
    return (float(score_scale) * (k @ q)).astype(np.float32)


# ---------------------------------------------------------------- top-p (Eq. 5)
def softmax_mass(s: np.ndarray):
    """Row maximum M, normaliser Z = sum exp(s - M) and probabilities (fp64)."""
    s64 = np.asarray(s, dtype=np.float64)
    M = float(np.max(s64))
    e = np.exp(s64 - M)
    Z = float(np.sum(e))
    return M, Z, e / Z


def descending_order(s: np.ndarray) -> np.ndarray:
    """Token ids by decreasing score; equal scores keep the smaller id first."""
    s64 = np.asarray(s, dtype=np.float64)
    return np.argsort(-s64, kind="stable")


def topp_select(s: np.ndarray, p: float):
    """Top-P(s, p) of Eq. 5 on the fp32 scores of one query row.

    Returns (ids ascending, k_star, mass of the set, threshold score, order,
    cumulative mass along the order).  k_star is the smallest k >= 1 whose
    prefix mass is >= p; p >= 1 keeps every key.
    """
    if not (p > 0.0):
        raise ValueError("top_p must be in (0, 1]")
    s = np.asarray(s, dtype=np.float32)
    n = s.shape[0]
    if n == 0:
        raise ValueError("empty row")
    _, _, P = softmax_mass(s)
    order = descending_order(s)
    cum = np.cumsum(P[order])
    if p >= 1.0:
        k_star = n
    else:
        hit = np.nonzero(cum >= p)[0]
        k_star = int(hit[0]) + 1 if hit.size else n
    ids = np.sort(order[:k_star])
    return ids, k_star, float(cum[k_star - 1]), float(s[order[k_star - 1]]), order, cum


def classify_against_band(s: np.ndarray, p: float, band: float = 1e-4):
    """Mandatory / optional / forbidden tokens for comparing a selection that was
    produced with fp32 mass sums: a token whose cumulative mass *before* its own
    inclusion lies within ``band`` of p may go either way."""
    ids, k_star, mass, thr, order, cum = topp_select(s, p)
    before = np.concatenate([[0.0], cum[:-1]])
    mandatory = order[before < p - band]
    forbidden = order[before >= p + band]
    if p >= 1.0:
        mandatory, forbidden = order, order[:0]
    return set(mandatory.tolist()), set(forbidden.tolist())


def set_mass(s: np.ndarray, ids) -> float:
    """Softmax mass (over the whole row) carried by the tokens ``ids``."""
    _, _, P = softmax_mass(s)
    return float(np.sum(P[np.asarray(sorted(ids), dtype=np.int64)]))


# ---------------------------------------------------------------- fixed-budget variant (Section 4.1)
def topk_select(s: np.ndarray, k: int):
    """The fixed-budget selector the paper compares against in Section 4.1 (k = 4096
    there): the k keys with the largest scores, equal scores going to the smaller
    position; every key when the row has no more than k.  Returns (ids ascending,
    number taken, threshold score = the smallest score taken, largest position taken
    among the keys that have the threshold score)."""
    if k < 1:
        raise ValueError("top_k must be >= 1")
    s = np.asarray(s, dtype=np.float32)
    n = s.shape[0]
    if n == 0:
        raise ValueError("empty row")
    order = descending_order(s)
    c = min(int(k), n)
    taken = order[:c]
    thr = float(s[taken[-1]])
    tie_last = int(max(int(i) for i in taken if s[i] == s[taken[-1]]))
    return np.sort(taken), c, thr, tie_last


def forced_tokens(m: int, n_sink: int, n_recent: int) -> np.ndarray:
    """Positions a variant may force into the set of query position m whatever their
    scores: the first n_sink keys and the n_recent newest ones (m itself included),
    restricted to the causal range [0, m]."""
    n = m + 1
    head = np.arange(0, min(max(n_sink, 0), n), dtype=np.int64)
    tail = np.arange(max(0, n - max(n_recent, 0)), n, dtype=np.int64)
    return np.union1d(head, tail)


def with_forced(ids, m: int, n_sink: int, n_recent: int) -> np.ndarray:
    """Union of a selected set with the forced positions (ascending)."""
    return np.union1d(np.asarray(ids, dtype=np.int64), forced_tokens(m, n_sink, n_recent))


# ---------------------------------------------------------------- block-wise top-p (Section 3.4)
def block_lse(s: np.ndarray, block: int = 64):
    """Per-block log-sum-exp pairs of one row's scores (Section 3.4): block b holds keys
    b*block .. min((b+1)*block, n) - 1; m_b is its largest score (as fp32) and
    l_b = sum exp(s - m_b) over its keys (fp64)."""
    s = np.asarray(s, dtype=np.float32)
    n = s.shape[0]
    if n == 0:
        raise ValueError("empty row")
    n_b = (n + block - 1) // block
    m = np.empty(n_b, dtype=np.float32)
    l = np.empty(n_b, dtype=np.float64)
    for b in range(n_b):
        blk = s[b * block: (b + 1) * block].astype(np.float64)
        m[b] = np.float32(blk.max())
        l[b] = np.sum(np.exp(blk - float(m[b])))
    return m, l


def topp_select_blocks(s: np.ndarray, p: float, block: int = 64):
    """Block-wise Top-P of Section 3.4 on the fp32 scores of one query row.

    Blocks are ordered by decreasing m_b (equal maxima: smaller block first); the
    selection is the shortest prefix of that order whose mass, sum of
    l_b exp(m_b - M) / Z, reaches p; p >= 1 keeps every block.  Returns
    (selected block ids ascending, their number, mass of the selection, m_b of the
    last block taken, order, cumulative mass along the order)."""
    if not (p > 0.0):
        raise ValueError("top_p must be in (0, 1]")
    m, l = block_lse(s, block)
    M = float(m.max())
    w = l * np.exp(m.astype(np.float64) - M)
    P = w / float(np.sum(w))
    order = np.argsort(-m.astype(np.float64), kind="stable")
    cum = np.cumsum(P[order])
    n_b = m.shape[0]
    if p >= 1.0:
        k_star = n_b
    else:
        hit = np.nonzero(cum >= p)[0]
        k_star = int(hit[0]) + 1 if hit.size else n_b
    ids = np.sort(order[:k_star])
    return ids, k_star, float(cum[k_star - 1]), float(m[order[k_star - 1]]), order, cum


def classify_blocks_against_band(s: np.ndarray, p: float, block: int = 64, band: float = 1e-4):
    """Mandatory / forbidden blocks for comparing a block selection made with fp32 mass
    sums: a block whose cumulative mass before its own inclusion lies within ``band`` of p
    may go either way."""
    ids, k_star, mass, thr, order, cum = topp_select_blocks(s, p, block)
    before = np.concatenate([[0.0], cum[:-1]])
    mandatory = order[before < p - band]
    forbidden = order[before >= p + band]
    if p >= 1.0:
        mandatory, forbidden = order, order[:0]
    return set(mandatory.tolist()), set(forbidden.tolist())


def block_token_set(block_ids, m: int, block: int = 64) -> np.ndarray:
    """Token positions 0..m covered by the given blocks."""
    n = np.arange(m + 1, dtype=np.int64)
    keep = np.zeros((m + block) // block + 1, dtype=bool)
    keep[np.asarray(sorted(block_ids), dtype=np.int64)] = True
    return n[keep[n // block]]


# ---------------------------------------------------------------- token sets
def dense_set(m: int) -> np.ndarray:
    return np.arange(m + 1, dtype=np.int64)


def local_set(m: int, n_sink: int, window: int) -> np.ndarray:
    """Sinks {0..n_sink-1} united with the window (m-W, m], clipped to 0..m."""
    n = np.arange(m + 1, dtype=np.int64)
    return n[(n < n_sink) | (n > m - window)]


# ---------------------------------------------------------------- Eq. 5: attention
def attention_over_set(q_bf16: np.ndarray, k_bf16: np.ndarray, v_bf16: np.ndarray,
                       ids, sm_scale: float):
    """Exact attention of one query over the keys ``ids`` (Eq. 5).

    q_bf16 [128]; k_bf16, v_bf16 [L, 128] (one KV head).  Returns
    (out float64 [128], log-sum-exp of the scaled logits over the set).
    """
    ids = np.asarray(ids, dtype=np.int64)
    q = bf16_to_f64(q_bf16)
    k = bf16_to_f64(k_bf16[ids])
    v = bf16_to_f64(v_bf16[ids])
    logit = (k @ q) * float(sm_scale)
    mx = float(np.max(logit))
    w = np.exp(logit - mx)
    z = float(np.sum(w))
    out = (w / z) @ v
    return out, mx + np.log(z)


# ---------------------------------------------------------------- whole rows
def retrieval_row(q_pre_bf16, q_bf16, w_q_bf16, kt_bf16, k_bf16, v_bf16, m: int,
                  p: float, score_scale: float, sm_scale: float):
    """One retrieval query head at position m: indexer -> top-p -> attention.

    kt_bf16: projected index keys [>= m+1, 16] of the head's index head;
    k_bf16/v_bf16: [>= m+1, 128] of its KV head.
    """
    qt = index_project(q_pre_bf16, w_q_bf16)
    s = index_scores(qt, kt_bf16[: m + 1], score_scale)
    ids, k_star, mass, thr, _, _ = topp_select(s, p)
    out, lse = attention_over_set(q_bf16, k_bf16, v_bf16, ids, sm_scale)
    return {"qt": qt, "scores": s, "ids": ids, "count": k_star, "mass": mass,
            "thresh": thr, "out": out, "lse": lse}


def local_row(q_bf16, k_bf16, v_bf16, m: int, n_sink: int, window: int, sm_scale: float):
    return attention_over_set(q_bf16, k_bf16, v_bf16, local_set(m, n_sink, window), sm_scale)


def dense_row(q_bf16, k_bf16, v_bf16, m: int, sm_scale: float):
    return attention_over_set(q_bf16, k_bf16, v_bf16, dense_set(m), sm_scale)
