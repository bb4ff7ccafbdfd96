"""CPU oracle for QuoKA's per-chunk sparse prefill attention.

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and
the benchmark's CPU-baseline leg may import this module.  It shares nothing with
the CUDA path: no kernels, headers, helpers or tables, and neither side imports
the other.

Everything here is plain numpy in float64, written step by step in the order and
notation of the paper (Algorithm 1 "KV cache sub-selection", Algorithm 2 "Chunked
prefill", Eq. 1-3).  No blocking, no fusion, no reordering.  All functions work on
ONE sequence (the batch axis is a loop in the caller):

    q        (n_Q,  C, d)      the chunk's queries            Q_i
    k, v     (n_KV, T+C, d)    rows [0,T) = cache K_<i, V_<i; rows [T,T+C) = K_i, V_i

Symbols: C = B_CP (chunk length), N = min(N_Q, C) retained queries,
B = min(B_SA, T) key budget, G = n_Q / n_KV.

Readings of the paper that this file fixes (each one is pinned by a CPU test):
  * Alg. 1 keeps the N_Q queries with the LOWEST cosine to the mean query
    (topk of the negated similarity), listed most-dissimilar first; equal
    cosines keep the earlier chunk position first.
  * The mean query is the per-head mean over chunk positions of the
    un-normalised queries.
  * The reshape/mean over the G heads of a KV group pairs the heads' retained
    queries BY RANK (the j-th retained query of every head), and head h belongs
    to KV head h // G.
  * Q-bar is not re-normalised: a score is a mean of cosines.
  * Normalised keys are used for scoring only; attention (Alg. 2, Eq. 2) runs on
    the original K and V.
  * Only cached keys (rows < T) are scored and budgeted; the chunk's own keys
    are always attended, causally, diagonal included.
  * top-B ties: the lower position wins; the index list is reported ascending.
  * Norms are clamped below by EPS.

Parity status: no function is "parity unpinned" in the sense of lacking a test
against something other than itself, but the paper prints no numeric worked
example of Algorithm 1, so the rank-pairing reading above is pinned only
structurally (linearity of the group mean, and G = 1 reducing to plain
max-cosine).
"""
from __future__ import annotations

import numpy as np

EPS = 1e-12


# --------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------
def round_to_bf16(x):
    """Round float values to the nearest bfloat16 (ties to even) and return them
    as float64.  bfloat16 = the upper 16 bits of an IEEE float32, so rounding is
    done on the float32 bit pattern: add 0x7FFF plus the lowest kept bit, then
    clear the low 16 bits.  Inputs are first rounded to float32, the type the
    value is held in before it is stored."""
    f = np.asarray(x, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32).astype(np.float64)
    # NaN / inf pass through unchanged in value class
    out = np.where(np.isfinite(f), out, f.astype(np.float64))
    return out


def key_budget(T, kv_budget, budget_frac):
    """B for one sequence.  kv_budget > 0: B = min(B_SA, T).  Otherwise the
    budget is a fraction of the cached length, rounded to nearest:
    B = floor(frac * T + 0.5), clipped to [0, T]."""
    T = int(T)
    if kv_budget is not None and kv_budget > 0:
        return min(int(kv_budget), T)
    B = int(np.floor(float(np.float32(budget_frac)) * T + 0.5))
    return max(0, min(B, T))


# --------------------------------------------------------------------------
# Algorithm 1, "Query Sub-selection"
# --------------------------------------------------------------------------
def query_cosines(q):
    """S_Q = CosSim(Q, M_Q) with M_Q = mean(Q, dim=positions), per head.
    q: (n_Q, C, d) -> (n_Q, C)."""
    q = np.asarray(q, dtype=np.float64)
    M = q.mean(axis=1)                                        # (n_Q, d)
    qn = np.maximum(np.sqrt((q * q).sum(axis=2)), EPS)        # (n_Q, C)
    Mn = np.maximum(np.sqrt((M * M).sum(axis=1)), EPS)        # (n_Q,)
    dots = np.einsum("hcd,hd->hc", q, M)
    return dots / (qn * Mn[:, None])


def select_queries(q, n_retain):
    """If C > N_Q keep topk(-S_Q, N_Q): the N_Q lowest cosines, most dissimilar
    first, ties to the earlier position.  Otherwise keep every query in position
    order.  Returns (q_idx (n_Q, N) int32 ordered, S_Q (n_Q, C))."""
    q = np.asarray(q, dtype=np.float64)
    n_q, C, _ = q.shape
    cos = query_cosines(q)
    if C > n_retain:
        order = np.argsort(cos, axis=1, kind="stable")        # ascending cosine
        q_idx = order[:, :n_retain]
    else:
        q_idx = np.tile(np.arange(C), (n_q, 1))
    return q_idx.astype(np.int32), cos


# --------------------------------------------------------------------------
# Algorithm 1, "Efficient Cosine Similarity via Pre-aggregation"
# --------------------------------------------------------------------------
def aggregate_queries(q, q_idx, n_kv, storage="f32", score_mode="cosine"):
    """Q <- gather(Q, idx); Q <- Q / norm(Q); Q-bar <- mean over the G heads of
    each KV group of the rank-aligned retained queries.  (n_KV, N, d).
    With storage == "bf16" Q-bar is rounded once to bfloat16, because it is
    stored in the cache dtype before the scoring product.
    score_mode == "dot" is the ablation of the Appendix "Ablations" (dot
    products instead of cosine similarity): the division by the norm is left
    out, everything else is unchanged."""
    q = np.asarray(q, dtype=np.float64)
    n_q, C, d = q.shape
    G = n_q // n_kv
    assert G * n_kv == n_q
    N = q_idx.shape[1]
    gathered = np.take_along_axis(q, q_idx.astype(np.int64)[:, :, None], axis=1)  # (n_Q, N, d)
    assert score_mode in ("cosine", "dot")
    if score_mode == "cosine":
        norms = np.maximum(np.sqrt((gathered * gathered).sum(axis=2, keepdims=True)), EPS)
        q_hat = gathered / norms
    else:
        q_hat = gathered
    qbar = q_hat.reshape(n_kv, G, N, d).mean(axis=1)
    if storage == "bf16":
        qbar = round_to_bf16(qbar)
    return qbar


def key_inv_norms(k):
    """1 / max(|k_t|, EPS) for every cache row.  Alg. 1 recomputes the key norms in every chunk; a caller may
    keep these instead (a cached key never changes).  k: (n_KV, rows, d) -> (n_KV, rows)."""
    k = np.asarray(k, dtype=np.float64)
    return 1.0 / np.maximum(np.sqrt((k * k).sum(axis=2)), EPS)


def score_keys(qbar, k, T, score_mode="cosine", query_agg="max", k_inv_norm=None):
    """K <- K / norm(K); S <- Q-bar K^T; S-hat <- max(S, dim=queries).
    qbar: (n_KV, N, d); k: (n_KV, >=T, d).  Returns (n_KV, T).
    The two ablations of the Appendix "Ablations": score_mode == "dot" leaves
    the keys un-normalised; query_agg == "mean" takes the mean over the query
    axis instead of the maximum."""
    assert score_mode in ("cosine", "dot") and query_agg in ("max", "mean")
    qbar = np.asarray(qbar, dtype=np.float64)
    kc = np.asarray(k, dtype=np.float64)[:, :T, :]
    if score_mode == "cosine" and k_inv_norm is not None:
        k_hat = kc * np.asarray(k_inv_norm, dtype=np.float64)[:, :T, None]     # cached 1/|k| instead of a fresh norm
    elif score_mode == "cosine":
        kn = np.maximum(np.sqrt((kc * kc).sum(axis=2, keepdims=True)), EPS)
        k_hat = kc / kn
    else:
        k_hat = kc
    S = qbar @ np.swapaxes(k_hat, 1, 2)                       # (n_KV, N, T)
    if S.shape[1] == 0:
        return np.full((kc.shape[0], T), -np.inf)
    return S.max(axis=1) if query_agg == "max" else S.mean(axis=1)


def select_keys(scores, B):
    """I <- topk(S-hat, B) per KV head: the B largest scores, ties to the lower
    position; reported ascending by position.  scores: (n_KV, T) -> (n_KV, B)."""
    scores = np.asarray(scores, dtype=np.float64)
    n_kv, T = scores.shape
    B = min(int(B), T)
    out = np.zeros((n_kv, B), dtype=np.int32)
    for h in range(n_kv):
        order = np.argsort(-scores[h], kind="stable")         # descending, earlier first on ties
        out[h] = np.sort(order[:B])
    return out


# --------------------------------------------------------------------------
# Eq. 1-2 and Algorithm 2: attention over [selected cache | causal chunk]
# --------------------------------------------------------------------------
def _attend(qh, kh, vh, T, idx, scale):
    """One query head.  qh (C, d); kh, vh (T+C, d); idx: selected cached rows."""
    C, d = qh.shape
    K_act = np.concatenate([kh[idx], kh[T:T + C]], axis=0)    # [K-hat | K_i]
    V_act = np.concatenate([vh[idx], vh[T:T + C]], axis=0)
    logits = (qh @ K_act.T) * scale                           # (C, B + C)
    nb = len(idx)
    r = np.arange(C)[:, None]
    u = np.arange(C)[None, :]
    mask = np.zeros_like(logits)
    mask[:, nb:] = np.where(u <= r, 0.0, -np.inf)             # causal inside the chunk
    logits = logits + mask
    m = logits.max(axis=1, keepdims=True)
    p = np.exp(logits - m)
    s = p.sum(axis=1, keepdims=True)
    out = (p / s) @ V_act
    lse = (m + np.log(s))[:, 0]
    return out, lse


def sparse_attention(q, k, v, T, k_idx, scale=None):
    """Y_i = Attention(Q_i, [K-hat | K_i], [V-hat | V_i]) with K-hat, V-hat the
    rows k_idx[kv] of the ORIGINAL cache.  q (n_Q, C, d); k, v (n_KV, >=T+C, d);
    k_idx: sequence of n_KV index arrays.  Returns (out (n_Q, C, d), lse (n_Q, C))."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n_q, C, d = q.shape
    n_kv = k.shape[0]
    G = n_q // n_kv
    if scale is None or scale == 0:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((n_q, C, d))
    lse = np.zeros((n_q, C))
    for h in range(n_q):
        kv = h // G
        idx = np.asarray(k_idx[kv], dtype=np.int64)
        out[h], lse[h] = _attend(q[h], k[kv], v[kv], T, idx, scale)
    return out, lse


def dense_chunk_attention(q, k, v, T, scale=None):
    """Eq. 2: the chunk attends every cached key and its own keys causally."""
    n_kv = np.asarray(k).shape[0]
    return sparse_attention(q, k, v, T, [np.arange(T)] * n_kv, scale)


def sparse_attention_rows(q, k, v, T, k_idx, heads, rows, scale=None):
    """The same attention for sampled (head, row) pairs only, one by one.
    Returns (len(heads), d).  Used at sizes where the full output is too slow."""
    q = np.asarray(q)
    n_q, C, d = q.shape
    n_kv = np.asarray(k).shape[0]
    G = n_q // n_kv
    if scale is None or scale == 0:
        scale = 1.0 / np.sqrt(d)
    res = np.zeros((len(heads), d))
    for i, (h, r) in enumerate(zip(heads, rows)):
        kv = h // G
        idx = np.asarray(k_idx[kv], dtype=np.int64)
        rows_u = np.concatenate([idx, np.arange(T, T + r + 1)])
        kk = np.asarray(k[kv][rows_u], dtype=np.float64)
        vv = np.asarray(v[kv][rows_u], dtype=np.float64)
        logit = (kk @ np.asarray(q[h, r], dtype=np.float64)) * scale
        p = np.exp(logit - logit.max())
        res[i] = (p / p.sum()) @ vv
    return res


# --------------------------------------------------------------------------
# the whole per-chunk path
# --------------------------------------------------------------------------
def quoka_prefill_chunk(q, k, v, T, n_retain, kv_budget=0, budget_frac=0.0,
                        storage="f32", scale=None, score_mode="cosine", query_agg="max"):
    """Algorithm 2, loop body, for one sequence: select queries, score and select
    cached keys, attend.  Returns a dict with every intermediate."""
    n_kv = np.asarray(k).shape[0]
    T = int(T)
    B = key_budget(T, kv_budget, budget_frac)
    q_idx, cos = select_queries(q, n_retain)
    qbar = aggregate_queries(q, q_idx, n_kv, storage, score_mode)
    scores = score_keys(qbar, k, T, score_mode, query_agg)
    k_idx = select_keys(scores, B)
    out, lse = sparse_attention(q, k, v, T, k_idx, scale)
    return dict(q_idx=q_idx, cos=cos, qbar=qbar, scores=scores, k_idx=k_idx,
                out=out, lse=lse, B=B)
