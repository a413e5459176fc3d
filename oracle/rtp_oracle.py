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
* ``attention_over_set`` Eq. 5, softmax(q.k/sqrt(d_h)) restricted to S, times V.
* ``local_set``          Section 3.2 / Table 2: attention sinks plus a sliding
                         window on local heads.
* ``dense_set``          ordinary causal attention (what retrieval heads do in
                         the paper's prefill; the in-library comparator).

Readings taken where the paper is silent (each also listed in the design notes):
no extra scale inside the top-p softmax; ties broken towards the smaller token
index; p = 1 keeps every causal key; the selection is never empty; sinks, the
recent window and the query's own position are NOT forced into a retrieval
head's set; a query at position m sees keys 0..m; the window is the last W
positions including m; query head h reads KV head h // G.

Pins (tests/test_oracle_*.py): brute force over all subsets for tiny L, closed
forms (equal scores, geometric scores, one dominant score, Gaussian scores),
shift / permutation / monotonicity invariants, dense attention against
torch's scaled_dot_product_attention, boolean-mask SDPA for the local pattern,
and the matrix-product identity for the indexer.  The selection statistics the
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
