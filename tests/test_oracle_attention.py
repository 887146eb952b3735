"""Pins for the oracle's attention step (Eq. 3) and its merges (CPU only)."""
import math

import numpy as np
import torch

from oracle import lsa_oracle as orc


def _problem(rng, L, H, dqk, dv):
    q = rng.standard_normal((L, H, dqk))
    k = rng.standard_normal((L, dqk))
    v = rng.standard_normal((L, dv))
    return q, k, v


def test_full_budget_equals_dense_causal_attention_from_library():
    """Ksp >= t: S_t = [0, t], so Eq. 3 is textbook causal softmax attention."""
    rng = np.random.default_rng(0)
    L, H, dqk, dv, S, W = 48, 3, 16, 8, 2, 5
    q, k, v = _problem(rng, L, H, dqk, dv)
    scale = 1 / math.sqrt(dqk)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                       # [1, H, L, d]
    tk = torch.from_numpy(k)[None, None].expand(1, H, L, dqk)
    tv = torch.from_numpy(v)[None, None].expand(1, H, L, dv)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)[0]
    for t in range(L):
        sparse = np.arange(S, max(S, t - W + 1))                           # every candidate selected
        S_t = orc.index_set(t, S, W, sparse)
        assert sorted(S_t) == list(range(t + 1))
        out, lse = orc.attend(q[t], k, v, S_t, scale)
        assert np.abs(out - ref[:, t].numpy()).max() < 1e-12
        z = scale * (q[t] @ k[:t + 1].T)
        assert np.abs(lse - torch.logsumexp(torch.from_numpy(z), dim=1).numpy()).max() < 1e-12


def test_no_sparse_budget_equals_band_masked_attention():
    """Ksp = 0: sink + sliding window = dense attention under the matching mask."""
    rng = np.random.default_rng(1)
    L, H, dqk, dv, S, W = 40, 2, 8, 8, 3, 6
    q, k, v = _problem(rng, L, H, dqk, dv)
    scale = 0.3
    tt, ss = np.meshgrid(np.arange(L), np.arange(L), indexing="ij")
    mask = (ss <= tt) & ((ss < S) | (ss > tt - W))
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k)[None, None].expand(1, H, L, dqk)
    tv = torch.from_numpy(v)[None, None].expand(1, H, L, dv)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask), scale=scale)[0]
    for t in range(L):
        out, _ = orc.attend(q[t], k, v, orc.index_set(t, S, W, []), scale)
        assert np.abs(out - ref[:, t].numpy()).max() < 1e-12


def test_one_key_and_uniform_cases():
    rng = np.random.default_rng(2)
    q, k, v = _problem(rng, 10, 2, 4, 3)
    out, lse = orc.attend(q[0], k, v, [7], 0.5)
    assert np.allclose(out, np.broadcast_to(v[7], (2, 3))) and np.allclose(lse, 0.5 * q[0] @ k[7])
    # zero query: uniform weights -> mean of the values, lse = log n
    out, lse = orc.attend(np.zeros((2, 4)), k, v, [1, 4, 6, 9], 1.0)
    assert np.allclose(out, v[[1, 4, 6, 9]].mean(axis=0)) and np.allclose(lse, math.log(4))


def test_two_branch_merge_equals_joint_softmax_and_order_is_irrelevant():
    """Sparse branch and sink+window branch merged by log-sum-exp rescaling = one softmax
    (the equivalence the hybrid operator of Sec. 4.1.1 and the sharded decode of App. B rely on)."""
    rng = np.random.default_rng(3)
    L, H, dqk, dv, S, W = 200, 4, 16, 8, 4, 30
    q, k, v = _problem(rng, L, H, dqk, dv)
    t = 180
    sparse = np.sort(rng.permutation(np.arange(S, t - W + 1))[:40])
    S_t = orc.index_set(t, S, W, sparse)
    joint, lse = orc.attend(q[t], k, v, S_t, 0.25)
    fixed = orc.index_set(t, S, W, [])
    o1, l1 = orc.attend(q[t], k, v, sparse, 0.25)
    o2, l2 = orc.attend(q[t], k, v, fixed, 0.25)
    om, lm = orc.merge_partials([o1, o2], [l1, l2])
    assert np.abs(om - joint).max() < 1e-12 and np.abs(lm - lse).max() < 1e-12
    # three shards dealt by page (i mod 3)
    parts = [S_t[(S_t // 16) % 3 == r] for r in range(3)]
    res = [orc.attend(q[t], k, v, p, 0.25) for p in parts]
    om, lm = orc.merge_partials([r[0] for r in res], [r[1] for r in res])
    assert np.abs(om - joint).max() < 1e-12
    perm, _ = orc.attend(q[t], k, v, rng.permutation(S_t), 0.25)
    assert np.abs(perm - joint).max() < 1e-12


def test_mla_value_is_prefix_of_latent_and_paged_gather():
    rng = np.random.default_rng(4)
    n, dqk, dv, page = 100, 12, 8, 16
    kv = rng.standard_normal((n, dqk))
    q = rng.standard_normal((2, dqk))
    S_t = np.array([0, 1, 17, 40, 99])
    out, _ = orc.attend(q, kv, kv[:, :dv], S_t, 0.2)
    # explicit weights
    z = 0.2 * q @ kv[S_t].T
    p = np.exp(z) / np.exp(z).sum(axis=1, keepdims=True)
    assert np.allclose(out, p @ kv[S_t][:, :dv]) and np.allclose(p.sum(axis=1), 1.0)
    # paged: scatter the logical rows into a shuffled pool, read back through the table
    n_pages = -(-n // page)
    table = rng.permutation(n_pages + 3)[:n_pages]
    pool = np.full(((n_pages + 3) * page, dqk), np.nan)
    for s in range(n):
        pool[table[s // page] * page + s % page] = kv[s]
    assert np.array_equal(orc.gather_paged(pool, table, n, page), kv)
    assert list(orc.paged_rows([0, 17, 99], table, page)) == [table[0] * 16, table[1] * 16 + 1, table[6] * 16 + 3]


def test_layer_group_reuses_one_index_set():
    rng = np.random.default_rng(5)
    L, H_I, d_I, H, dqk, dv = 120, 2, 4, 2, 8, 4
    qI = rng.standard_normal((L, H_I, d_I)); w = rng.standard_normal((L, H_I)); kI = rng.standard_normal((L, d_I))
    km = orc.block_means(kI, 4)
    qs = [rng.standard_normal((H, dqk)) for _ in range(3)]
    ks = [rng.standard_normal((L, dqk)) for _ in range(3)]
    vs = [x[:, :dv] for x in ks]
    t = 110
    kw = dict(P=16, B=4, M=2, Ksp=10, S=2, W=12)
    sparse, pages, outs, lses = orc.layer_group_query(t, qI[t], w[t], kI, km, qs, ks, vs, sm_scale=0.3, **kw)
    sp2, _ = orc.select_sparse(t, qI[t], w[t], kI, km, **kw)
    assert list(sparse) == list(sp2) and len(outs) == 3
    for r in range(3):
        o, l = orc.attend(qs[r], ks[r], vs[r], orc.index_set(t, 2, 12, sparse), 0.3)
        assert np.array_equal(o, outs[r]) and np.array_equal(l, lses[r])
