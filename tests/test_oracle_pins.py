"""Pins for the CPU oracle: each test checks an oracle function against something
the paper or the mathematics fixes (a hand-derived example, a closed form, a
library routine for a special case, brute force, an invariant), never against the
oracle's own formula retyped.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest
import torch
from scipy.spatial.distance import cdist

from oracle import quoka_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alg1_2d_example.txt")


def rng(seed):
    return np.random.default_rng(seed)


def rand_problem(seed, n_q=4, n_kv=2, C=8, T=12, d=4):
    r = rng(seed)
    q = r.normal(size=(n_q, C, d)) + r.normal(size=(n_q, 1, d))
    k = r.normal(size=(n_kv, T + C, d))
    v = r.normal(size=(n_kv, T + C, d))
    return q, k, v


# ------------------------------------------------------------------ storage rounding
def test_bf16_rounding_known_values():
    # 1 + 2^-8 is exactly half-way between 1 and 1 + 2^-7: ties to even -> 1
    assert O.round_to_bf16(1.0 + 2.0 ** -8) == 1.0
    # 1 + 3*2^-8 is half-way between 1+2^-7 (odd) and 1+2^-6 (even) -> 1 + 2^-6
    assert O.round_to_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6
    assert O.round_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert O.round_to_bf16(-0.3) == float(torch.tensor(-0.3).to(torch.bfloat16))
    assert O.round_to_bf16(0.0) == 0.0


def test_bf16_rounding_matches_library_cast():
    x = rng(0).normal(size=20000).astype(np.float32) * np.float32(3.0)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_to_bf16(x), want)


def test_budget_fraction_reproduces_stated_budgets():
    # 12 % of 32768 and of 131072 cached keys, as the benchmark configurations state them
    assert O.key_budget(32768, 0, 0.12) == 3932
    assert O.key_budget(131072, 0, 0.12) == 15729
    assert O.key_budget(100, 512, 0.0) == 100      # B = min(B_SA, T)
    assert O.key_budget(0, 512, 0.0) == 0


# ------------------------------------------------------------------ hand-derived 2-D example
def _load_golden():
    vals = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#") or line.startswith("["):
            continue
        name, rhs = line.split("=")
        vals[name.strip()] = np.array([float(t) for t in rhs.split()])
    return vals


def test_algorithm1_hand_example():
    g = _load_golden()
    q = np.stack([g["q_head0"].reshape(4, 2), g["q_head1"].reshape(4, 2)])
    k = g["k"].reshape(1, 4, 2)
    q_idx, cos = O.select_queries(q, 2)
    np.testing.assert_allclose(cos[0], g["cos_head0"], atol=1e-12)
    np.testing.assert_allclose(cos[1], g["cos_head1"], atol=1e-12)
    # q0 and q1 have equal cosines analytically; rounding may order them either way, the
    # lowest (q3) is unambiguous and the second must be one of the tied pair
    assert q_idx[0, 0] == 3 and q_idx[1, 0] == 3
    assert q_idx[0, 1] in (0, 1) and q_idx[1, 1] in (0, 1)
    q_idx = np.stack([g["q_idx_head0"], g["q_idx_head1"]]).astype(np.int32)
    qbar = O.aggregate_queries(q, q_idx, n_kv=1)
    np.testing.assert_allclose(qbar.reshape(-1), g["qbar"], atol=1e-12)
    scores = O.score_keys(qbar, k, 4)
    np.testing.assert_allclose(scores[0], g["scores"], atol=1e-9)
    # k0, k1, k2 tie at 0.5 analytically; force the exact tie so the tie rule itself is tested
    s = np.array([[0.5, 0.5, 0.5, g["scores"][3]]])
    np.testing.assert_array_equal(O.select_keys(s, 2)[0], g["k_idx_B2"])
    np.testing.assert_array_equal(O.select_keys(s, 3)[0], g["k_idx_B3"])
    # one head alone (G = 1): plain max-cosine
    qbar1 = O.aggregate_queries(q[:1], q_idx[:1], n_kv=1)
    s1 = O.score_keys(qbar1, k, 4)
    np.testing.assert_allclose(s1[0], g["scores_head0_alone"], atol=1e-9)
    np.testing.assert_array_equal(O.select_keys(np.array([[1.0, 0.0, 1.0, 0.5]]), 2)[0],
                                  g["k_idx_head0_alone_B2"])


def test_ablation_variants_hand_example_and_invariants():
    """Dot-product scoring and mean-over-queries aggregation (Appendix "Ablations")."""
    g = _load_golden()
    q = np.stack([g["q_head0"].reshape(4, 2), g["q_head1"].reshape(4, 2)])
    k = g["k"].reshape(1, 4, 2)
    q_idx = np.stack([g["q_idx_head0"], g["q_idx_head1"]]).astype(np.int32)
    # head 0 alone, raw dot products: table values
    qb = O.aggregate_queries(q[:1], q_idx[:1], n_kv=1, score_mode="dot")
    np.testing.assert_allclose(qb[0], q[0][[3, 0]], atol=0)              # raw retained rows, no normalisation
    np.testing.assert_allclose(O.score_keys(qb, k, 4, "dot", "max")[0], g["dot_max_head0_alone"], atol=1e-9)
    np.testing.assert_allclose(O.score_keys(qb, k, 4, "dot", "mean")[0], g["dot_mean_head0_alone"], atol=1e-9)
    # both heads, cosine scoring, mean over the two ranks
    qbar = O.aggregate_queries(q, q_idx, n_kv=1)
    np.testing.assert_allclose(O.score_keys(qbar, k, 4, "cosine", "mean")[0], g["cos_mean"], atol=1e-9)
    # invariants on random data: dot scores are linear in the key, cosine scores ignore its length;
    # mean <= max; one retained query makes mean == max; dot/max with G = 1 is a plain matrix product
    qr, kr, _ = rand_problem(5, n_q=4, n_kv=2, C=9, d=8, T=13)
    idx, _ = O.select_queries(qr, 3)
    for mode in ("cosine", "dot"):
        qb = O.aggregate_queries(qr, idx, 2, score_mode=mode)
        mx = O.score_keys(qb, kr, 13, mode, "max")
        mn = O.score_keys(qb, kr, 13, mode, "mean")
        assert (mn <= mx + 1e-12).all()
        k2 = kr.copy()
        k2[:, 5] *= 3.0
        mx2 = O.score_keys(qb, k2, 13, mode, "max")
        want = mx.copy()
        if mode == "dot":
            want[:, 5] *= 3.0
        np.testing.assert_allclose(mx2, want, atol=1e-12)
        one = O.score_keys(qb[:, :1], kr, 13, mode, "mean")
        np.testing.assert_allclose(one, O.score_keys(qb[:, :1], kr, 13, mode, "max"), atol=1e-12)
    idx1 = np.tile(np.arange(9), (4, 1)).astype(np.int32)                 # all queries, G = 1
    qb = O.aggregate_queries(qr, idx1, 4, score_mode="dot")
    dots = np.stack([qr[h] @ kr[h // 2, :13].T for h in range(4)])        # (4, C, T), written out per head
    kr4 = np.stack([kr[h // 2] for h in range(4)])
    got = O.score_keys(qb, kr4, 13, "dot", "max")
    np.testing.assert_allclose(got, dots.max(axis=1), atol=1e-12)


def test_cached_inverse_key_norms_hand_values_and_equivalence():
    g = _load_golden()
    k = g["k"].reshape(1, 4, 2)
    # |k| = 3, 5, 2*sqrt(2), 2 for the hand example's keys
    np.testing.assert_allclose(O.key_inv_norms(k)[0], [1 / 3, 0.2, 1 / (2 * np.sqrt(2)), 0.5], atol=1e-15)
    q, kr, _ = rand_problem(6, n_q=4, n_kv=2, C=9, d=8, T=13)
    idx, _ = O.select_queries(q, 3)
    qb = O.aggregate_queries(q, idx, 2)
    inv = O.key_inv_norms(kr)
    np.testing.assert_allclose(inv, 1.0 / np.linalg.norm(kr, axis=2), rtol=1e-14)
    for agg in ("max", "mean"):
        np.testing.assert_allclose(O.score_keys(qb, kr, 13, "cosine", agg, k_inv_norm=inv),
                                   O.score_keys(qb, kr, 13, "cosine", agg), atol=1e-14)
    # the cache is used as given: a stale entry changes exactly that key's score, by the ratio
    stale = inv.copy()
    stale[:, 4] *= 2.0
    a = O.score_keys(qb, kr, 13, k_inv_norm=stale)
    b = O.score_keys(qb, kr, 13)
    np.testing.assert_allclose(a[:, 4], 2.0 * b[:, 4], atol=1e-14)
    np.testing.assert_allclose(np.delete(a, 4, axis=1), np.delete(b, 4, axis=1), atol=1e-14)
    # dot-product scoring ignores it; a zero key gets the clamped inverse, not infinity
    np.testing.assert_allclose(O.score_keys(qb, kr, 13, "dot", k_inv_norm=stale), O.score_keys(qb, kr, 13, "dot"), atol=0)
    assert np.isfinite(O.key_inv_norms(np.zeros((1, 2, 4)))).all()


# ------------------------------------------------------------------ query sub-selection
def test_query_cosines_match_library_cosine_distance():
    q, _, _ = rand_problem(1, n_q=3, C=17, d=8)
    cos = O.query_cosines(q)
    for h in range(3):
        want = 1.0 - cdist(q[h], q[h].mean(axis=0, keepdims=True), metric="cosine")[:, 0]
        np.testing.assert_allclose(cos[h], want, atol=1e-12)


def test_lowest_cosine_queries_are_kept_most_dissimilar_first():
    r = rng(2)
    C, d, N = 32, 16, 5
    base = r.normal(size=d)
    q = base[None, :] + 0.1 * r.normal(size=(C, d))
    M0 = q.mean(axis=0)
    q[7] = -4.0 * M0        # anti-aligned with the mean: must be retained first
    q[11] = 9.0 * q.mean(axis=0)   # (nearly) parallel to the mean: must not be retained
    idx, cos = O.select_queries(q[None], N)
    assert idx.shape == (1, N)
    assert idx[0, 0] == 7
    assert 11 not in idx[0]
    kept = cos[0][idx[0]]
    assert np.all(np.diff(kept) >= 0)                       # ascending cosine = most dissimilar first
    others = np.delete(cos[0], idx[0])
    assert kept.max() <= others.min()
    # against a library argsort of a library cosine distance (largest distance first)
    dist = cdist(q, q.mean(axis=0, keepdims=True), metric="cosine")[:, 0]
    np.testing.assert_array_equal(idx[0], np.argsort(-dist, kind="stable")[:N])


def test_two_queries_have_equal_cosine_to_their_mean():
    # closed form: with C = 2 the mean bisects... only when lengths are equal; in general
    # cos(q_a, M) and cos(q_b, M) satisfy |q_a| c_a = (|q_a|^2 + q_a.q_b)/(2|M|): check that identity
    r = rng(3)
    q = r.normal(size=(1, 2, 6))
    cos = O.query_cosines(q)[0]
    a, b = q[0]
    M = 0.5 * (a + b)
    for vec, c in ((a, cos[0]), (b, cos[1])):
        assert abs(np.linalg.norm(vec) * c - (vec @ vec + a @ b) / (2 * np.linalg.norm(M))) < 1e-12
    # equal lengths -> the mean bisects the angle -> equal cosines
    b2 = b * np.linalg.norm(a) / np.linalg.norm(b)
    c2 = O.query_cosines(np.stack([a, b2])[None])[0]
    assert abs(c2[0] - c2[1]) < 1e-12


def test_no_selection_when_chunk_not_longer_than_n_retain():
    q, _, _ = rand_problem(4, n_q=2, C=6)
    for N in (6, 9):
        idx, _ = O.select_queries(q, N)
        np.testing.assert_array_equal(idx, np.tile(np.arange(6), (2, 1)))


def test_theorem1_bound_holds_for_oracle_cosines():
    # Theorem 1: CosSim(k,q0) = beta > 0 and CosSim(M_Q,k) = alpha < 0 imply
    # CosSim(M_Q, q0) <= 1 + alpha*beta - alpha^2/2 - beta^2/2.
    r = rng(5)
    hits = 0
    for _ in range(300):
        q = r.normal(size=(1, 6, 3))
        k = r.normal(size=3)
        M = q[0].mean(axis=0)
        alpha = 1 - cdist(M[None], k[None], metric="cosine")[0, 0]
        cos = O.query_cosines(q)[0]
        for j in range(6):
            beta = 1 - cdist(q[0, j][None], k[None], metric="cosine")[0, 0]
            if beta > 0 and alpha < 0:
                hits += 1
                assert cos[j] <= 1 + alpha * beta - 0.5 * alpha ** 2 - 0.5 * beta ** 2 + 1e-12
    assert hits > 100


# ------------------------------------------------------------------ scoring and aggregation
def post_aggregation_scores(q, q_idx, k, T, n_kv):
    """Per-head cosine scores first (library cosine distance), mean over the G heads
    of the group afterwards, then max over the retained rank: the order of operations
    the method's pre-aggregation is claimed to be equal to."""
    n_q = q.shape[0]
    G = n_q // n_kv
    N = q_idx.shape[1]
    out = np.zeros((n_kv, T))
    for kv in range(n_kv):
        per_head = np.zeros((G, N, T))
        for gq in range(G):
            h = kv * G + gq
            per_head[gq] = 1.0 - cdist(q[h][q_idx[h]], k[kv][:T], metric="cosine")
        out[kv] = per_head.mean(axis=0).max(axis=0)
    return out


@pytest.mark.parametrize("n_q,n_kv", [(4, 2), (8, 2), (3, 3), (8, 1)])
def test_pre_aggregation_equals_post_aggregation(n_q, n_kv):
    q, k, _ = rand_problem(6, n_q=n_q, n_kv=n_kv, C=10, T=23, d=8)
    q_idx, _ = O.select_queries(q, 4)
    qbar = O.aggregate_queries(q, q_idx, n_kv)
    got = O.score_keys(qbar, k, 23)
    want = post_aggregation_scores(q, q_idx, k, 23, n_kv)
    np.testing.assert_allclose(got, want, atol=1e-12)
    assert np.all(np.abs(got) <= 1 + 1e-12)


def test_rank_pairing_uses_each_heads_own_order():
    # two heads in one group retain DIFFERENT positions in different orders; Q-bar_j must
    # average the heads' j-th retained queries, not queries at equal positions
    q = np.zeros((2, 3, 2))
    q[0] = [[1, 0], [0, 1], [1, 1]]
    q[1] = [[0, 2], [3, 0], [1, 1]]
    q_idx = np.array([[2, 0], [1, 0]], dtype=np.int32)
    qbar = O.aggregate_queries(q, q_idx, n_kv=1)
    s = np.sqrt(0.5)
    np.testing.assert_allclose(qbar[0, 0], [(s + 1) / 2, (s + 0) / 2], atol=1e-12)
    np.testing.assert_allclose(qbar[0, 1], [(1 + 0) / 2, (0 + 1) / 2], atol=1e-12)


def test_contiguous_head_grouping():
    # heads 0,1 -> KV head 0; heads 2,3 -> KV head 1
    q, k, _ = rand_problem(7, n_q=4, n_kv=2, C=5, T=9, d=4)
    q_idx, _ = O.select_queries(q, 5)
    qbar = O.aggregate_queries(q, q_idx, 2)
    qn = q / np.linalg.norm(q, axis=2, keepdims=True)
    np.testing.assert_allclose(qbar[0], 0.5 * (qn[0] + qn[1]), atol=1e-12)
    np.testing.assert_allclose(qbar[1], 0.5 * (qn[2] + qn[3]), atol=1e-12)


def test_qbar_bf16_is_single_rounding():
    q, _, _ = rand_problem(8, n_q=4, n_kv=2, C=6, d=8)
    q_idx, _ = O.select_queries(q, 3)
    exact = O.aggregate_queries(q, q_idx, 2, "f32")
    rounded = O.aggregate_queries(q, q_idx, 2, "bf16")
    want = torch.from_numpy(exact.astype(np.float32)).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(rounded, want)


def test_zero_key_scores_zero():
    q, k, _ = rand_problem(9, n_q=2, n_kv=1, C=4, T=5, d=4)
    k[0, 2] = 0.0
    q_idx, _ = O.select_queries(q, 2)
    s = O.score_keys(O.aggregate_queries(q, q_idx, 1), k, 5)
    assert np.isfinite(s).all() and s[0, 2] == 0.0


# ------------------------------------------------------------------ key selection
def test_top_b_is_the_max_sum_subset_bruteforce():
    r = rng(10)
    for T, B in [(7, 3), (9, 4), (6, 6), (8, 1)]:
        s = r.normal(size=(1, T))
        got = O.select_keys(s, B)[0]
        best = max(itertools.combinations(range(T), B), key=lambda c: s[0, list(c)].sum())
        np.testing.assert_array_equal(got, np.array(best))
        assert np.all(np.diff(got) > 0)


def test_top_b_ties_keep_lower_position():
    s = np.array([[0.3, 0.9, 0.3, 0.3, 0.1]])
    np.testing.assert_array_equal(O.select_keys(s, 3)[0], [0, 1, 2])
    np.testing.assert_array_equal(O.select_keys(s, 2)[0], [0, 1])
    np.testing.assert_array_equal(O.select_keys(s, 9)[0], [0, 1, 2, 3, 4])   # B > T -> all


# ------------------------------------------------------------------ attention
def sdpa_reference(q, k, v, T, visible_cached):
    """torch's scaled_dot_product_attention (a library routine) with an explicit boolean
    mask: cached column t visible iff visible_cached[kv][t]; chunk column u visible to row r iff u <= r."""
    n_q, C, d = q.shape
    n_kv = k.shape[0]
    G = n_q // n_kv
    out = np.zeros_like(q)
    for h in range(n_q):
        kv = h // G
        mask = torch.zeros(C, T + C, dtype=torch.bool)
        mask[:, :T] = torch.from_numpy(np.asarray(visible_cached[kv]))[None, :]
        mask[:, T:] = torch.tril(torch.ones(C, C, dtype=torch.bool))
        o = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[h])[None], torch.from_numpy(k[kv, :T + C])[None],
            torch.from_numpy(v[kv, :T + C])[None], attn_mask=mask[None])
        out[h] = o[0].numpy()
    return out


def test_dense_chunk_attention_matches_library_sdpa():
    q, k, v = rand_problem(11, n_q=4, n_kv=2, C=9, T=14, d=8)
    got, _ = O.dense_chunk_attention(q, k, v, 14)
    want = sdpa_reference(q, k, v, 14, [np.ones(14, bool)] * 2)
    np.testing.assert_allclose(got, want, atol=1e-12)


def test_sparse_attention_matches_library_sdpa_with_selected_mask():
    q, k, v = rand_problem(12, n_q=4, n_kv=2, C=7, T=20, d=8)
    idx = [np.array([1, 4, 5, 19]), np.array([0, 2, 3, 11])]
    vis = []
    for a in idx:
        m = np.zeros(20, bool)
        m[a] = True
        vis.append(m)
    got, _ = O.sparse_attention(q, k, v, 20, idx)
    np.testing.assert_allclose(got, sdpa_reference(q, k, v, 20, vis), atol=1e-12)


def test_full_budget_and_all_queries_equals_dense():
    q, k, v = rand_problem(13, n_q=4, n_kv=2, C=8, T=16, d=8)
    res = O.quoka_prefill_chunk(q, k, v, 16, n_retain=8, kv_budget=16)
    want = sdpa_reference(q, k, v, 16, [np.ones(16, bool)] * 2)
    np.testing.assert_allclose(res["out"], want, atol=1e-12)
    res2 = O.quoka_prefill_chunk(q, k, v, 16, n_retain=3, kv_budget=999)   # B_SA > T
    np.testing.assert_allclose(res2["out"], want, atol=1e-12)


def test_empty_cache_is_causal_self_attention_and_row0_is_v0():
    q, k, v = rand_problem(14, n_q=2, n_kv=1, C=5, T=0, d=4)
    res = O.quoka_prefill_chunk(q, k, v, 0, n_retain=2, kv_budget=4)
    np.testing.assert_allclose(res["out"][:, 0], np.broadcast_to(v[0, 0], (2, 4)), atol=1e-12)
    want = sdpa_reference(q, k, v, 0, [np.zeros(0, bool)])
    np.testing.assert_allclose(res["out"], want, atol=1e-12)


def test_identical_keys_give_uniform_average_of_visible_values():
    # closed form: equal logits -> softmax is uniform over the visible set
    r = rng(15)
    T, C, d = 10, 4, 4
    q = r.normal(size=(1, C, d))
    k = np.tile(r.normal(size=(1, 1, d)), (1, T + C, 1))
    v = r.normal(size=(1, T + C, d))
    idx = [np.array([2, 3, 7])]
    out, lse = O.sparse_attention(q, k, v, T, idx)
    for row in range(C):
        vis = np.concatenate([v[0, idx[0]], v[0, T:T + row + 1]])
        np.testing.assert_allclose(out[0, row], vis.mean(axis=0), atol=1e-12)
        logit = (q[0, row] @ k[0, 0]) / np.sqrt(d)
        assert abs(lse[0, row] - (logit + np.log(3 + row + 1))) < 1e-12


def test_softmax_rows_sum_to_one_via_lse():
    q, k, v = rand_problem(16, n_q=2, n_kv=1, C=6, T=11, d=4)
    idx = [np.array([0, 5, 9])]
    _, lse = O.sparse_attention(q, k, v, 11, idx)
    for h in range(2):
        for r_ in range(6):
            rows = np.concatenate([idx[0], np.arange(11, 11 + r_ + 1)])
            logits = k[0, rows] @ q[h, r_] / 2.0
            assert abs(np.exp(logits - lse[h, r_]).sum() - 1.0) < 1e-12


def test_attention_uses_original_keys_not_normalised_ones():
    # scaling one selected key changes the output (it would not if normalised keys were used)
    q, k, v = rand_problem(17, n_q=2, n_kv=1, C=3, T=6, d=4)
    idx = [np.array([1, 4])]
    a, _ = O.sparse_attention(q, k, v, 6, idx)
    k2 = k.copy()
    k2[0, 4] *= 3.0
    b, _ = O.sparse_attention(q, k2, v, 6, idx)
    assert np.abs(a - b).max() > 1e-3
    np.testing.assert_allclose(b, sdpa_reference(q, k2, v, 6, [np.isin(np.arange(6), idx[0])]), atol=1e-12)


def test_sampled_rows_agree_with_full_output():
    q, k, v = rand_problem(18, n_q=4, n_kv=2, C=6, T=9, d=4)
    idx = [np.array([0, 3]), np.array([2, 8])]
    full, _ = O.sparse_attention(q, k, v, 9, idx)
    heads, rows = [0, 3, 2], [5, 0, 2]
    got = O.sparse_attention_rows(q, k, v, 9, idx, heads, rows)
    for i, (h, r_) in enumerate(zip(heads, rows)):
        np.testing.assert_allclose(got[i], full[h, r_], atol=1e-12)


# ------------------------------------------------------------------ invariances of the whole path
def test_selection_invariant_to_positive_rescaling():
    q, k, v = rand_problem(19, n_q=4, n_kv=2, C=8, T=30, d=8)
    a = O.quoka_prefill_chunk(q, k, v, 30, n_retain=3, kv_budget=7)
    r = rng(20)
    q2 = q * r.uniform(0.5, 4.0)            # a common positive factor keeps the mean direction
    k2 = k.copy()
    k2[:, :30] *= r.uniform(0.2, 5.0, size=(2, 30, 1))   # any per-key positive factor
    b = O.quoka_prefill_chunk(q2, k2, v, 30, n_retain=3, kv_budget=7)
    np.testing.assert_array_equal(a["q_idx"], b["q_idx"])
    np.testing.assert_allclose(a["scores"], b["scores"], atol=1e-12)
    np.testing.assert_array_equal(a["k_idx"], b["k_idx"])


def test_permuting_cached_positions_permutes_selection_and_keeps_output():
    q, k, v = rand_problem(21, n_q=4, n_kv=2, C=5, T=24, d=8)
    T = 24
    a = O.quoka_prefill_chunk(q, k, v, T, n_retain=3, kv_budget=6)
    perm = rng(22).permutation(T)
    k2, v2 = k.copy(), v.copy()
    k2[:, :T] = k[:, perm]
    v2[:, :T] = v[:, perm]
    b = O.quoka_prefill_chunk(q, k2, v2, T, n_retain=3, kv_budget=6)
    for kv in range(2):
        assert set(perm[b["k_idx"][kv]].tolist()) == set(a["k_idx"][kv].tolist())
    np.testing.assert_allclose(a["out"], b["out"], atol=1e-12)


def test_index_set_shape_and_range():
    q, k, v = rand_problem(23, n_q=4, n_kv=2, C=5, T=24, d=8)
    res = O.quoka_prefill_chunk(q, k, v, 24, n_retain=3, budget_frac=0.25)
    assert res["B"] == 6 and res["k_idx"].shape == (2, 6)
    for kv in range(2):
        a = res["k_idx"][kv]
        assert len(set(a.tolist())) == 6 and a.min() >= 0 and a.max() < 24


# ------------------------------------------------------------------ planted mistakes must be caught
MUTANTS = {
    "keep highest cosine": ('order = np.argsort(cos, axis=1, kind="stable")', 'order = np.argsort(-cos, axis=1, kind="stable")'),
    "mean over queries": ("return S.max(axis=1)", "return S.mean(axis=1)"),
    "interleaved head grouping": ("q_hat.reshape(n_kv, G, N, d).mean(axis=1)", "q_hat.reshape(G, n_kv, N, d).mean(axis=0)"),
    "normalise mean query first": ("M = q.mean(axis=1) ", "M = (q / np.sqrt((q*q).sum(axis=2, keepdims=True))).mean(axis=1) "),
    "dot product scoring": ("k_hat = kc / kn", "k_hat = kc"),
    "diagonal excluded": ("np.where(u <= r, 0.0, -np.inf)", "np.where(u < r, 0.0, -np.inf)"),
    "no softmax scale": ("scale = 1.0 / np.sqrt(d)", "scale = 1.0"),
    "lowest scores selected": ("order = np.argsort(-scores[h], kind=\"stable\")", "order = np.argsort(scores[h], kind=\"stable\")"),
    "ties to higher position": ("order = np.argsort(-scores[h], kind=\"stable\")", "order = (len(scores[h]) - 1 - np.argsort(-scores[h][::-1], kind=\"stable\"))"),
    "wrong kv head for attention": ("        kv = h // G\n        idx = np.asarray(k_idx[kv], dtype=np.int64)\n        out[h]", "        kv = h % n_kv\n        idx = np.asarray(k_idx[kv], dtype=np.int64)\n        out[h]"),
    "renormalised qbar": ("    if storage == \"bf16\":\n        qbar = round_to_bf16(qbar)\n    return qbar", "    qbar = qbar / np.sqrt((qbar*qbar).sum(axis=2, keepdims=True))\n    return qbar"),
    "truncating bf16": ("rounded = (bits + np.uint64(0x7FFF) + lsb)", "rounded = (bits)"),
    "dot mode normalises keys": ("    else:\n        k_hat = kc", "    else:\n        k_hat = kc / np.sqrt((kc * kc).sum(axis=2, keepdims=True))"),
    "dot mode normalises queries": ("    else:\n        q_hat = gathered", "    else:\n        q_hat = gathered / np.sqrt((gathered * gathered).sum(axis=2, keepdims=True))"),
    "mean mode sums": ("else S.mean(axis=1)", "else S.sum(axis=1)"),
    "cached norm used as a norm": ("k_hat = kc * np.asarray(k_inv_norm", "k_hat = kc / np.asarray(k_inv_norm"),
    "inverse norm of the squared norm": ("return 1.0 / np.maximum(np.sqrt((k * k).sum(axis=2)), EPS)", "return 1.0 / np.maximum((k * k).sum(axis=2), EPS)"),
}

PIN_TESTS = [
    test_bf16_rounding_known_values, test_algorithm1_hand_example,
    test_lowest_cosine_queries_are_kept_most_dissimilar_first,
    test_two_queries_have_equal_cosine_to_their_mean,
    lambda: test_pre_aggregation_equals_post_aggregation(8, 2),
    test_contiguous_head_grouping, test_top_b_is_the_max_sum_subset_bruteforce,
    test_top_b_ties_keep_lower_position, test_dense_chunk_attention_matches_library_sdpa,
    test_empty_cache_is_causal_self_attention_and_row0_is_v0,
    test_identical_keys_give_uniform_average_of_visible_values,
    test_full_budget_and_all_queries_equals_dense, test_query_cosines_match_library_cosine_distance,
    test_selection_invariant_to_positive_rescaling, test_ablation_variants_hand_example_and_invariants,
    test_cached_inverse_key_norms_hand_values_and_equivalence,
]


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, monkeypatch):
    """Plant one plausible mistake in a copy of the oracle and require a pin to fail."""
    import types

    old, new = MUTANTS[name]
    src = open(O.__file__).read()
    assert src.count(old) >= 1, f"mutation site for '{name}' not found"
    mutated = types.ModuleType("oracle_mutant")
    mutated.__file__ = O.__file__
    exec(compile(src.replace(old, new), "oracle_mutant", "exec"), mutated.__dict__)
    g = globals()
    monkeypatch.setitem(g, "O", mutated)
    caught = False
    for t in PIN_TESTS:
        try:
            t()
        except AssertionError:
            caught = True
            break
        except Exception:
            caught = True
            break
    assert caught, f"no pin noticed the planted mistake: {name}"
