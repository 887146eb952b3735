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
