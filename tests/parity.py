"""Helpers that compare the CUDA path with the CPU oracle stage by stage.

The path is checked as a chain: each stage's CUDA output is validated against the
oracle within that stage's tie rule, then the CUDA output itself (not the
oracle's) is fed to the oracle's next stage.  Index work is bit-exact up to ties:
a rank or a key may differ from the oracle's only where the oracle's own score
gap is below 1e-4 relative.  Attention outputs on identical indices: bf16 within
2e-2 max-abs (outputs up to 3.1 in magnitude; see attention_bound for larger ones)
and 2e-3 mean-abs; f32 within 2e-4 / 2e-5.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import quoka_oracle as O
from paper_2602_08722_b200 import api

REL_TIE = 1e-4
SCORE_ATOL = 2e-5
ATTN_TOL = {"bf16": (2e-2, 2e-3), "f32": (2e-4, 2e-5)}


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def check_query_ranks(q_idx_gpu: np.ndarray, cos: np.ndarray, n_retain: int):
    """q_idx_gpu (n_Q, N), cos (n_Q, C) from the oracle."""
    n_q, C = cos.shape
    if C <= n_retain:
        np.testing.assert_array_equal(q_idx_gpu, np.tile(np.arange(C), (n_q, 1)))
        return 0
    swaps = 0
    for h in range(n_q):
        g = q_idx_gpu[h].astype(np.int64)
        assert len(set(g.tolist())) == len(g) and g.min() >= 0 and g.max() < C
        order = np.argsort(cos[h], kind="stable")
        want = order[:n_retain]
        tau = cos[h][order[n_retain - 1]]
        tol = REL_TIE * abs(tau)
        chosen = np.zeros(C, bool)
        chosen[g] = True
        assert chosen[cos[h] < tau - tol].all(), "a clearly dissimilar query was not retained"
        assert not chosen[cos[h] > tau + tol].any(), "a clearly similar query was retained"
        cg = cos[h][g]
        gaps = np.diff(cg)
        assert (gaps >= -REL_TIE * np.abs(cg[1:]) - 1e-12).all(), "retained queries out of rank order"
        swaps += int((g != want).sum())
    return swaps


def check_qbar(qbar_gpu: np.ndarray, qbar_oracle: np.ndarray, dtype: str):
    diff = np.abs(qbar_gpu - qbar_oracle)
    if dtype == "bf16":
        # one bf16 ulp is at most 2^-7 relative; entries that nearly cancel carry the fp32 accumulation
        # error of their O(0.1) terms (a few 1e-8) on top, which near zero exceeds their own ulp
        ulp = np.abs(qbar_oracle) * 2.0 ** -7 + 2e-7
        assert (diff <= ulp).all(), f"Qbar differs by more than one bf16 ulp (max excess {(diff - ulp).max()})"
        assert (diff > 0).mean() < 0.01, "too many Qbar entries rounded differently"
    else:
        assert diff.max() <= 1e-6, f"Qbar max abs diff {diff.max()}"


def check_key_selection(k_idx_gpu: np.ndarray, scores_oracle: np.ndarray, B: int):
    """k_idx_gpu (n_KV, >=B); scores_oracle (n_KV, T)."""
    n_kv, T = scores_oracle.shape
    diffs = 0
    for kv in range(n_kv):
        g = k_idx_gpu[kv, :B].astype(np.int64)
        assert len(g) == B
        if B == 0:
            continue
        assert (np.diff(g) > 0).all(), "selected rows not ascending / not unique"
        assert g.min() >= 0 and g.max() < T
        s = scores_oracle[kv]
        want = O.select_keys(s[None], B)[0]
        tau = np.sort(s)[::-1][B - 1]
        tol = REL_TIE * abs(tau)
        chosen = np.zeros(T, bool)
        chosen[g] = True
        assert chosen[s > tau + tol].all(), "a key clearly above the threshold was dropped"
        assert not chosen[s < tau - tol].any(), "a key clearly below the threshold was selected"
        diffs += int(B - np.intersect1d(g, want).size)
    return diffs


def attention_bound(out_oracle: np.ndarray, dtype: str) -> np.ndarray:
    """Element-wise bound on |out_gpu - out_oracle|.

    f32: 2e-4 everywhere.  bf16: the stated 2e-2 max-abs, or, where it is larger, what the arithmetic costs at
    that magnitude: the output is STORED in bf16, so rounding the exact result alone may cost half a bf16 spacing
    of |o| (0.0078 for 2 <= |o| < 4, 0.0156 for 4 <= |o| < 8), and the softmax weights enter the PV product as
    bf16 (2^-9 relative each; on a row that few keys dominate they do not average out, and the row sum is taken
    before the rounding), which adds up to 2^-8 |o|.  The sum exceeds 2e-2 from |o| = 3.12 on."""
    mx, _ = ATTN_TOL[dtype]
    a = np.abs(out_oracle)
    bound = np.full(a.shape, mx)
    if dtype == "bf16":
        spacing = np.ldexp(1.0, np.frexp(np.maximum(a, 1.0))[1] - 1 - 7)      # 2^(floor(log2 |o|) - 7), exactly
        bound = np.maximum(bound, spacing / 2 + a * 2.0 ** -8)
    return bound


def check_attention(out_gpu: np.ndarray, out_oracle: np.ndarray, dtype: str):
    """Returns the number of elements whose bound is above the stated 2e-2 (large outputs, bf16 only)."""
    diff = np.abs(out_gpu - out_oracle)
    _, mean = ATTN_TOL[dtype]
    assert np.isfinite(out_gpu).all()
    bound = attention_bound(out_oracle, dtype)
    worst = np.unravel_index(np.argmax(diff - bound), diff.shape)
    assert (diff <= bound).all(), (f"attention abs diff {diff[worst]} > {bound[worst]} at {worst} "
                                   f"(oracle value {out_oracle[worst]})")
    assert diff.mean() <= mean, f"attention mean abs diff {diff.mean()} > {mean}"
    return int((bound > ATTN_TOL[dtype][0]).sum()) if dtype == "bf16" else 0


class GpuProblem:
    """Device buffers + params for one ChunkInputs."""

    def __init__(self, inp, n_retain, kv_budget=0, budget_frac=0.0, impl=api.IMPL_AUTO, paged=False,
                 max_ctx_len=None, score_mode="cosine", query_agg="max", cached_norms=False):
        dev = "cuda"
        self.inp = inp
        self.dtype = inp.dtype
        self.q = inp.q.to(dev)
        if paged:
            self.k = inp.k_pages.to(dev)
            self.v = inp.v_pages.to(dev)
            self.block_table = inp.block_table.to(dev)
        else:
            self.k = inp.k.to(dev)
            self.v = inp.v.to(dev)
            self.block_table = None
        self.ctx_len = inp.ctx_len.to(dev)
        self.out = torch.zeros_like(self.q)
        b, n_q, C, d = self.q.shape
        n_kv = self.k.shape[1]
        self.b, self.n_q, self.n_kv, self.C, self.d = b, n_q, n_kv, C, d
        self.max_ctx = int(inp.ctx_len.max()) if max_ctx_len is None else int(max_ctx_len)
        self.n_retain, self.kv_budget, self.budget_frac = n_retain, kv_budget, budget_frac
        self.p = api.make_params(self.q, self.k, self.out, self.ctx_len, n_retain=n_retain, kv_budget=kv_budget,
                                 budget_frac=budget_frac, max_ctx_len=self.max_ctx, block_table=self.block_table,
                                 impl=impl, score_mode={"cosine": api.SCORE_COSINE, "dot": api.SCORE_DOT}[score_mode],
                                 query_agg={"max": api.AGG_MAX, "mean": api.AGG_MEAN}[query_agg])
        self.score_mode, self.query_agg = score_mode, query_agg
        self.N = min(n_retain, C)
        self.cap = api.quoka_kv_budget_cap(self.p)
        self.ws = api.alloc_workspace(self.p)
        self.q_idx = torch.full((b, n_q, self.N), -7, dtype=torch.int32, device=dev)
        self.qbar = torch.zeros((b, n_kv, self.N, d), dtype=self.q.dtype, device=dev)
        self.scores = torch.full((b, n_kv, max(self.max_ctx, 1)), float("nan"), dtype=torch.float32, device=dev)
        self.k_idx = torch.full((b, n_kv, self.cap), -7, dtype=torch.int32, device=dev)
        self.k_cnt = torch.full((b,), -7, dtype=torch.int32, device=dev)
        self.lse = torch.zeros((b, n_q, C), dtype=torch.float32, device=dev)
        self.k_inv_norm = None
        if cached_norms:
            # the cache of inverse key norms: built once for the rows already there, then kept per appended chunk
            self.k_inv_norm = torch.full(tuple(self.k.shape[:3]), float("nan"), dtype=torch.float32, device=dev)
            api.quoka_update_key_norms(self.p, self.k, self.k_inv_norm, True, self.ws)
            self.p.k_inv_norm = self.k_inv_norm.data_ptr()

    def run_staged(self):
        api.quoka_select_queries(self.p, self.q, self.q_idx, self.qbar, self.ws)
        api.quoka_score_keys(self.p, self.qbar, self.k, self.scores, self.ws)
        api.quoka_select_keys(self.p, self.scores, self.k_idx, self.k_cnt, self.ws)
        api.quoka_sparse_attn(self.p, self.q, self.k, self.v, self.k_idx, self.k_cnt, self.out, self.lse, self.ws)
        torch.cuda.synchronize()
        assert api.quoka_last_device_status(self.ws) == 0

    def oracle_inputs(self, s):
        T = int(self.inp.ctx_len[s])
        q = f64(self.inp.q[s])
        k = f64(self.inp.k[s, :, : T + self.C])
        v = f64(self.inp.v[s, :, : T + self.C])
        return q, k, v, T


def stratified_rows(n_q: int, C: int, n_random: int, seed: int):
    """(heads, rows) for a sampled attention check: for EVERY head the rows at the edges of the kernels' 128-row
    tiles (0, 127, 128, 255, 256, the last row, and the rows around the middle tile edge), then n_random uniformly
    drawn pairs."""
    mid = (C // 2) // 128 * 128
    edges = sorted({r for r in (0, 127, 128, 255, 256, mid - 1, mid, C - 129, C - 128, C - 1) if 0 <= r < C})
    heads = np.repeat(np.arange(n_q), len(edges))
    rows = np.tile(np.array(edges, dtype=np.int64), n_q)
    r = np.random.default_rng(seed)
    heads = np.concatenate([heads, r.integers(0, n_q, n_random)])
    rows = np.concatenate([rows, r.integers(0, C, n_random)])
    return heads, rows


def check_chain(gp: GpuProblem, attn_rows=None, seed=0):
    """Validate every stage of a staged run against the oracle.  attn_rows: number of randomly
    sampled (head, row) pairs per sequence for the attention check, on top of the tile-edge rows
    of every head (None = all rows)."""
    stats = dict(rank_swaps=0, key_diffs=0)
    for s in range(gp.b):
        q, k, v, T = gp.oracle_inputs(s)
        B = O.key_budget(T, gp.kv_budget, gp.budget_frac)
        assert int(gp.k_cnt[s]) == B
        # stage 1
        _, cos = O.select_queries(q, gp.n_retain)
        q_idx = gp.q_idx[s].cpu().numpy()
        stats["rank_swaps"] += check_query_ranks(q_idx, cos, gp.n_retain)
        # stage 2 on the GPU's ranks
        qbar_o = O.aggregate_queries(q, q_idx, gp.n_kv, gp.dtype, gp.score_mode)
        qbar_g = f64(gp.qbar[s])
        check_qbar(qbar_g, qbar_o, gp.dtype)
        # stage 3 on the GPU's Qbar
        if T > 0:
            # one KV head at a time: the oracle materialises the (N, T) score matrix
            sc_o = np.concatenate([O.score_keys(qbar_g[kv:kv + 1], k[kv:kv + 1], T, gp.score_mode, gp.query_agg)
                                   for kv in range(gp.n_kv)])
            sc_g = f64(gp.scores[s, :, :T])
            # raw dot products are not bounded by 1: the fp32 summation error scales with their magnitude
            atol = SCORE_ATOL * max(1.0, float(np.abs(sc_o).max()))
            assert np.abs(sc_g - sc_o).max() <= atol, f"score max abs diff {np.abs(sc_g - sc_o).max()}"
            if gp.score_mode == "cosine":
                assert np.abs(sc_g).max() <= 1 + 1e-5
        else:
            sc_o = np.zeros((gp.n_kv, 0))
        # stage 4: band rule against the oracle's scores
        k_idx = gp.k_idx[s].cpu().numpy()
        stats["key_diffs"] += check_key_selection(k_idx, sc_o, B)
        assert (k_idx[:, B:] == -1).all()
        # exact integer parity of the selection step on the GPU's own fp32 scores
        if T > 0:
            want = O.select_keys(f64(gp.scores[s, :, :T]), B)
            np.testing.assert_array_equal(k_idx[:, :B], want)
        # stage 5 on the GPU's indices
        idx_list = [k_idx[kv, :B] for kv in range(gp.n_kv)]
        out_g = f64(gp.out[s])
        if attn_rows is None:
            out_o, lse_o = O.sparse_attention(q, k, v, T, idx_list)
            stats["big_outputs"] = stats.get("big_outputs", 0) + check_attention(out_g, out_o, gp.dtype)
            assert np.abs(f64(gp.lse[s]) - lse_o).max() <= 2e-3
        else:
            heads, rows = stratified_rows(gp.n_q, gp.C, attn_rows, seed + s)
            out_o = O.sparse_attention_rows(q, k, v, T, idx_list, heads, rows)
            stats["big_outputs"] = stats.get("big_outputs", 0) + check_attention(out_g[heads, rows], out_o, gp.dtype)
    return stats
