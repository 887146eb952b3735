"""Pins for the oracle's scoring and selection steps (CPU only).

Each check compares the oracle with something written independently of it:
plain Python loops over the paper's formulas, a full sort, or an equivalence
the paper states.
"""
import math

import numpy as np
import pytest

from oracle import lsa_oracle as orc


def _rand_problem(rng, L, H, d, nonneg=False):
    q = rng.standard_normal((L, H, d)) / math.sqrt(d)
    k = rng.standard_normal((L, d)) / math.sqrt(d)
    w = rng.standard_normal((L, H)) / math.sqrt(H)
    if nonneg:
        q, k = np.abs(q), np.abs(k)
    return q, w, k


def _eq1_loops(q, w, k_s):
    """Eq. 1 for one (query, key) pair with scalar loops."""
    tot = 0.0
    for j in range(q.shape[0]):
        dot = 0.0
        for c in range(q.shape[1]):
            dot += q[j, c] * k_s[c]
        tot += w[j] * (dot if dot > 0 else 0.0)
    return tot


def _sorted_topk(pairs, k):
    """pairs = [(score, id)]: full sort by (score desc, id asc), cut, report ids ascending."""
    return sorted(i for _, i in sorted(pairs, key=lambda p: (-p[0], p[1]))[:k])


def test_indexer_scores_equal_scalar_loops():
    rng = np.random.default_rng(0)
    q, w, k = _rand_problem(rng, 24, 3, 5)
    got = orc.indexer_scores(q[7], w[7], k)
    for s in range(24):
        assert abs(got[s] - _eq1_loops(q[7], w[7], k[s])) < 1e-13
    # a transposed operand or a dropped ReLU would break this special case:
    # one head, weight 1, key = query  ->  score = |q|^2
    assert abs(orc.indexer_scores(q[3, :1], np.ones(1), q[3, :1])[0] - (q[3, 0] ** 2).sum()) < 1e-13
    # negative dot is clipped to zero
    assert orc.indexer_scores(q[3, :1], np.ones(1), -q[3, :1])[0] == 0.0


def test_page_scores_equal_scalar_loops():
    rng = np.random.default_rng(1)
    q, w, k = _rand_problem(rng, 70, 2, 4)
    P, B = 16, 4
    km = orc.block_means(k, B, round_bf16=False)
    got = orc.page_scores(q[60], w[60], km, P, B, [0, 2, 4])
    for g, p in zip(got, [0, 2, 4]):
        ref = 0.0
        for n in range(p * 4, min(p * 4 + 4, km.shape[0])):        # page 4 holds 64..69: 2 sub-blocks
            ref += _eq1_loops(q[60], w[60], km[n])
        assert abs(g - ref) < 1e-13


def test_page_score_linear_when_relu_inactive():
    """All dots >= 0: Eq. 9 equals (1/B) * sum of the page's token scores (Eq. 1 is then linear)."""
    rng = np.random.default_rng(2)
    q, w, k = _rand_problem(rng, 128, 4, 8, nonneg=True)
    P, B = 32, 8
    km = orc.block_means(k, B, round_bf16=False)
    for t in (40, 127):
        tok = orc.indexer_scores(q[t], w[t], k)
        pg = orc.page_scores(q[t], w[t], km, P, B, range(4))
        for p in range(4):
            assert abs(pg[p] - tok[p * P:(p + 1) * P].sum() / B) < 1e-12


def test_page_score_jensen_bound_and_B1_identity():
    rng = np.random.default_rng(3)
    q, w, k = _rand_problem(rng, 96, 4, 8)
    w = np.abs(w)                                   # w >= 0 makes the score convex in the key
    P = 32
    tok = orc.indexer_scores(q[90], w[90], k)
    for B in (2, 8, 32):
        pg = orc.page_scores(q[90], w[90], orc.block_means(k, B, round_bf16=False), P, B, range(3))
        for p in range(3):
            assert pg[p] <= tok[p * P:(p + 1) * P].sum() / B + 1e-12
    pg1 = orc.page_scores(q[90], w[90], orc.block_means(k, 1, round_bf16=False), P, 1, range(3))
    for p in range(3):
        assert abs(pg1[p] - tok[p * P:(p + 1) * P].sum()) < 1e-12


def test_top_k_equals_full_sort_with_heavy_ties_and_signed_zero():
    rng = np.random.default_rng(4)
    vals = np.array([0.0, -0.0, 1.5, -2.0], dtype=np.float32)
    for n, k in [(1, 1), (17, 5), (200, 64), (200, 200), (200, 300), (50, 0)]:
        scores = vals[rng.integers(0, 4, n)]
        ids = rng.permutation(1000)[:n]
        got = orc.top_k(scores, ids, k)
        assert list(got) == _sorted_topk([(float(s), int(i)) for s, i in zip(scores, ids)], k)
    # among equal scores the smaller id wins, whatever the order of presentation
    assert list(orc.top_k(np.zeros(6), np.array([9, 3, 7, 1, 5, 8]), 3)) == [1, 3, 5]
    assert list(orc.top_k(np.array([0.0, -0.0, 0.0, -0.0]), np.array([4, 2, 3, 1]), 2)) == [1, 2]


def test_top_k_decomposes_over_page_shards():
    """Local top-K on pages dealt round-robin to N ranks, then a re-rank of the K*N
    candidates, equals the global top-K (the sharded-cache decode of App. B)."""
    rng = np.random.default_rng(5)
    n, K, page, N = 1000, 50, 16, 4
    scores = np.round(rng.standard_normal(n), 1)          # coarse grid -> ties across shards
    ids = np.arange(n)
    cand = []
    for r in range(N):
        mine = ids[(ids // page) % N == r]
        cand.append(orc.top_k(scores[mine], mine, K))
    cand = np.concatenate(cand)
    assert list(orc.top_k(scores[cand], cand, K)) == list(orc.top_k(scores, ids, K))


def test_candidate_range_and_pages():
    assert orc.candidate_range(10, 4, 8) == (4, 2)                       # empty: hi < lo
    assert orc.eligible_pages(10, 4, 8, 16).size == 0
    assert list(orc.eligible_pages(12, 4, 8, 16)) == [0]                 # candidates {4}
    assert list(orc.eligible_pages(100, 4, 8, 16)) == [0, 1, 2, 3, 4, 5]  # candidates 4..92
    assert list(orc.eligible_pages(100, 16, 8, 16)) == [1, 2, 3, 4, 5]    # page 0 is all sink


@pytest.mark.parametrize("seed", range(6))
def test_hierarchical_equals_flat_brute_force_when_all_pages_kept(seed):
    """With M >= number of eligible pages the two-stage result must equal Eq. 7 computed
    by scoring every candidate with scalar loops and sorting them all."""
    rng = np.random.default_rng(10 + seed)
    L, H, d, P, B, S, W, Ksp = 150, 2, 4, 16, 4, 3, 20, 17
    q, w, k = _rand_problem(rng, L, H, d)
    km = orc.block_means(k, B)
    for t in [0, 2, 3, 22, 23, 24, 40, 41, 99, 149]:
        sparse, pages = orc.select_sparse(t, q[t], w[t], k, km, P=P, B=B, M=1000, Ksp=Ksp, S=S, W=W)
        flat = _sorted_topk([(_eq1_loops(q[t], w[t], k[s]), s) for s in range(S, t - W + 1)], Ksp)
        assert list(sparse) == flat
        flat2, _ = orc.select_sparse(t, q[t], w[t], k, km, P=P, B=B, M=2, Ksp=Ksp, S=S, W=W, hi_enable=False)
        assert list(flat2) == flat


def test_plain_dsa_special_case():
    """S = W = 0 and no hierarchy: Eq. 2, top-K over every s <= t."""
    rng = np.random.default_rng(20)
    q, w, k = _rand_problem(rng, 64, 2, 4)
    for t in (0, 5, 63):
        sparse, _ = orc.select_sparse(t, q[t], w[t], k, orc.block_means(k, 4), P=8, B=4, M=1, Ksp=6, S=0, W=0,
                                      hi_enable=False)
        assert list(sparse) == _sorted_topk([(_eq1_loops(q[t], w[t], k[s]), s) for s in range(t + 1)], 6)


@pytest.mark.parametrize("seed", range(4))
def test_two_stage_brute_force_with_real_recall(seed):
    """M smaller than the eligible page count: redo both stages with scalar loops."""
    rng = np.random.default_rng(30 + seed)
    L, H, d, P, B, S, W, M, Ksp = 200, 2, 4, 16, 4, 2, 24, 3, 20
    q, w, k = _rand_problem(rng, L, H, d)
    km = orc.block_means(k, B)
    for t in [60, 61, 120, 199]:
        lo, hi = S, t - W
        E = list(range(lo // P, hi // P + 1))
        ps = []
        for p in E:
            sc = 0.0
            for j in range(H):
                inner = 0.0
                for n in range(p * (P // B), min((p + 1) * (P // B), km.shape[0])):
                    dot = float(np.dot(q[t, j], km[n]))
                    inner += dot if dot > 0 else 0.0
                sc += w[t, j] * inner
            ps.append((sc, p))
        pages_ref = _sorted_topk(ps, M) if len(E) > M else E
        cand = [s for p in pages_ref for s in range(p * P, p * P + P) if lo <= s <= hi]
        ref = _sorted_topk([(_eq1_loops(q[t], w[t], k[s]), s) for s in cand], Ksp)
        sparse, pages = orc.select_sparse(t, q[t], w[t], k, km, P=P, B=B, M=M, Ksp=Ksp, S=S, W=W)
        assert list(pages) == pages_ref and list(sparse) == ref


def test_selection_invariants_and_index_set():
    rng = np.random.default_rng(40)
    L, H, d, P, B, S, W, M, Ksp = 300, 3, 8, 16, 8, 4, 32, 4, 40
    q, w, k = _rand_problem(rng, L, H, d)
    km = orc.block_means(k, B)
    for t in range(0, L, 7):
        sparse, pages = orc.select_sparse(t, q[t], w[t], k, km, P=P, B=B, M=M, Ksp=Ksp, S=S, W=W)
        E = orc.eligible_pages(t, S, W, P)
        assert len(pages) == min(M, len(E)) and set(pages) <= set(E)
        assert (np.diff(sparse) > 0).all()
        if sparse.size:
            assert sparse.min() >= S and sparse.max() <= t - W
            assert set(sparse // P) <= set(pages)
        n_cand = sum(min(t - W, p * P + P - 1) - max(S, p * P) + 1 for p in pages)
        assert sparse.size == min(Ksp, n_cand)
        S_t = orc.index_set(t, S, W, sparse)
        assert len(set(S_t)) == len(S_t) and S_t.max() <= t
        assert set(range(min(S, t + 1))) <= set(S_t) and set(range(max(0, t - W + 1), t + 1)) <= set(S_t)
        if t < S + W:
            assert list(S_t) == list(range(t + 1))


def test_coarse_stage_sees_whole_boundary_page_when_window_shorter_than_page():
    """W < P-1: an eligible page may reach past t; its mean keys still enter the coarse score
    (means are per cache, not per query), but no token beyond t-W is ever selected."""
    rng = np.random.default_rng(41)
    L, P, B = 96, 32, 8
    q, w, k = _rand_problem(rng, L, 2, 4)
    km = orc.block_means(k, B)
    t = 40                                                   # candidates 0..38, page 1 spans 32..63
    sparse, pages = orc.select_sparse(t, q[t], w[t], k, km, P=P, B=B, M=1, Ksp=64, S=0, W=2)
    ps = orc.page_scores(q[t], w[t], km, P, B, [0, 1])
    assert list(pages) == [0 if ps[0] >= ps[1] else 1]
    assert sparse.max() <= 38


def test_select_fp32_matches_sorted_reference_on_float32_compare():
    rng = np.random.default_rng(42)
    sc = rng.standard_normal(500).astype(np.float32)
    sc[::7] = sc[3]                                           # ties
    got = orc.select_fp32(sc, None, 400, 33, apply_range=True, S=4, W=50)
    assert list(got) == _sorted_topk([(float(sc[s]), s) for s in range(4, 351)], 33)
    pos = rng.permutation(2000)[:500].astype(np.int64)
    pos[::11] = -1
    got = orc.select_fp32(sc, pos, 0, 20, apply_range=False)
    assert list(got) == _sorted_topk([(float(s), int(p)) for s, p in zip(sc, pos) if p >= 0], 20)


# ---------------------------------------------------------------- MinMax pooling (Eq. 13)
def _eq13_loops(q, w, keys_of_page, B):
    """Eq. 13 page score with scalar loops over sub-blocks, heads and dimensions, extrema found token by token."""
    tot = 0.0
    n_tok = len(keys_of_page)
    for n0 in range(0, n_tok, B):
        blk = keys_of_page[n0:n0 + B]
        for j in range(q.shape[0]):
            s_tilde = 0.0
            for c in range(q.shape[1]):
                hi_c = max(float(k_s[c]) for k_s in blk)
                lo_c = min(float(k_s[c]) for k_s in blk)
                s_tilde += max(q[j, c] * hi_c, q[j, c] * lo_c)
            tot += w[j] * max(s_tilde, 0.0)
    return tot


def test_minmax_page_scores_equal_scalar_loops():
    rng = np.random.default_rng(31)
    P, B, H, d = 16, 4, 3, 8
    q, w, k = _rand_problem(rng, 70, H, d)             # 70 keys: the last page is partial, so is its last sub-block
    kmax, kmin = orc.block_minmax(k, B, round_bf16=False)
    pages = np.arange(-(-70 // P))
    got = orc.page_scores_minmax(q[5], w[5], kmax, kmin, P, B, pages)
    for p in pages:
        want = _eq13_loops(q[5], w[5], k[p * P:min((p + 1) * P, 70)], B)
        assert got[p] == pytest.approx(want, rel=1e-12, abs=1e-12)


def test_minmax_upper_bounds_every_token_score_and_B1_is_the_token_score():
    """s~ of Eq. 13 bounds q.k for every token of the sub-block from above (the reason the paper gives for it), so
    with non-negative head weights a page's MinMax score is at least the largest token score in it; with B = 1 the
    extrema are the key itself and MinMax, mean pooling and Eq. 1 coincide."""
    rng = np.random.default_rng(32)
    P, B, H, d = 8, 4, 2, 6
    q, w, k = _rand_problem(rng, 64, H, d)
    w = np.abs(w)
    kmax, kmin = orc.block_minmax(k, B, round_bf16=False)
    for n in range(kmax.shape[0]):
        s_tilde = np.maximum(q[9] * kmax[n], q[9] * kmin[n]).sum(axis=1)          # [H]
        for s in range(n * B, n * B + B):
            assert (s_tilde >= q[9] @ k[s] - 1e-12).all()
    pages = np.arange(64 // P)
    page_mm = orc.page_scores_minmax(q[9], w[9], kmax, kmin, P, B, pages)
    tok = orc.indexer_scores(q[9], w[9], k)
    for p in pages:
        assert page_mm[p] >= tok[p * P:(p + 1) * P].max() - 1e-12
    # B = 1
    k1max, k1min = orc.block_minmax(k, 1, round_bf16=False)
    assert np.array_equal(k1max, k) and np.array_equal(k1min, k)
    mm1 = orc.page_scores_minmax(q[9], w[9], k1max, k1min, P, 1, pages)
    mean1 = orc.page_scores(q[9], w[9], orc.block_means(k, 1, round_bf16=False), P, 1, pages)
    np.testing.assert_allclose(mm1, mean1, rtol=1e-12)
    np.testing.assert_allclose(mm1, tok.reshape(-1, P).sum(axis=1), rtol=1e-12)


def test_minmax_is_a_dot_product_of_split_queries():
    """max(q*a, q*b) with a >= b is q*a for q >= 0 and q*b for q < 0, so Eq. 13 is [q+ | q-] . [k_max | k_min]:
    the identity the GPU path computes with."""
    rng = np.random.default_rng(33)
    q, w, k = _rand_problem(rng, 32, 4, 8)
    kmax, kmin = orc.block_minmax(k, 8, round_bf16=False)
    qp, qm = np.maximum(q[3], 0.0), np.minimum(q[3], 0.0)
    for n in range(kmax.shape[0]):
        direct = np.maximum(q[3] * kmax[n], q[3] * kmin[n]).sum(axis=1)
        np.testing.assert_allclose(qp @ kmax[n] + qm @ kmin[n], direct, rtol=1e-12, atol=1e-15)


def test_minmax_selection_keeps_the_needle_page():
    """A page holding one key strongly aligned with the query is recalled by MinMax stage 1 even when the other keys
    of its sub-block are anti-aligned (a case where the mean cancels): the upper-bound property at work."""
    rng = np.random.default_rng(34)
    L, P, B, H, d = 512, 16, 8, 2, 16
    q, w, k = _rand_problem(rng, L, H, d)
    w = np.abs(w)
    t = L - 1
    needle = 100
    k[needle] = 6.0 * q[t, 0] / np.linalg.norm(q[t, 0])
    for s in range(96, 104):                     # the needle's sub-block: the others pull the mean the other way
        if s != needle:
            k[s] = -k[needle] / 7.0
    kw = dict(P=P, B=B, M=4, Ksp=32, S=2, W=8)
    mm = orc.block_minmax(k, B)
    sparse_mm, pages_mm = orc.select_sparse(t, q[t], w[t], k, None, minmax=mm, **kw)
    assert needle // P in pages_mm and needle in sparse_mm
    sparse_mean, pages_mean = orc.select_sparse(t, q[t], w[t], k, orc.block_means(k, B), **kw)
    assert needle // P not in pages_mean
