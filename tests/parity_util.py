"""Plumbing for the GPU parity tests: host copies of a workload and oracle runs on sampled queries."""
from __future__ import annotations

import numpy as np
import torch

from oracle import lsa_oracle as orc
from oracle import reference_run as ref

TOL_BF16 = dict(max_abs=2e-2, rel_l2=5e-3)
TOL_FP8 = dict(max_abs=5e-2, rel_l2=1e-2)
MIN_OVERLAP = 0.995          # mean over the checked queries (the end-to-end bar)
MIN_OVERLAP_ANY = 0.98       # no single query may fall below this (a near-tie flips a handful of its 2048 tokens at most)
MAX_PAGE_DIFF_SHARE = 0.02   # share of checked queries whose kept page set differs from the oracle's (near-tie at rank M)


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact host copy: bf16 -> float32, everything else unchanged."""
    t = t.detach()
    if t.dtype == torch.bfloat16:
        t = t.to(torch.float32)
    return t.cpu().numpy()


def boundary_queries(cfg, q_pos0, n_query, n_random, seed=0):
    """Query positions that exercise every regime change, plus a uniform random sample."""
    S, W, P, M = cfg.S, cfg.W, cfg.P, cfg.M
    t_m = (M + S // P) * P + W          # first query with more than M eligible pages
    pts = {0, S - 1, S, W - 1, W, S + W - 1, S + W, S + W + 1, t_m - 1, t_m, t_m + 1,
           t_m + P - 1, t_m + P, 2 * P + W - 1, 2 * P + W, q_pos0, q_pos0 + n_query - 1}
    rng = np.random.default_rng(seed)
    pts |= set(int(x) for x in rng.integers(q_pos0, q_pos0 + n_query, n_random))
    return sorted(t for t in pts if q_pos0 <= t < q_pos0 + n_query)


class Metrics:
    def __init__(self):
        self.overlaps, self.page_diff, self.max_abs, self.num, self.den = [], 0, 0.0, 0.0, 0.0
        self.lse_abs, self.n, self.n_pages = 0.0, 0, 0

    def add_select(self, gpu_sparse, ref_sparse, gpu_pages=None, ref_pages=None):
        self.overlaps.append(ref.overlap(gpu_sparse, ref_sparse))
        if gpu_pages is not None:
            self.n_pages += 1
            if list(gpu_pages) != list(ref_pages):
                self.page_diff += 1
        self.n += 1

    def add_out(self, gpu_out, ref_out, gpu_lse=None, ref_lse=None):
        d = gpu_out.astype(np.float64) - ref_out
        self.max_abs = max(self.max_abs, float(np.abs(d).max()))
        self.num += float((d * d).sum())
        self.den += float((ref_out * ref_out).sum())
        if gpu_lse is not None:
            self.lse_abs = max(self.lse_abs, float(np.abs(gpu_lse.astype(np.float64) - ref_lse).max()))

    @property
    def rel_l2(self):
        return (self.num / self.den) ** 0.5 if self.den > 0 else 0.0

    @property
    def mean_overlap(self):
        return float(np.mean(self.overlaps)) if self.overlaps else 1.0

    def summary(self):
        return dict(queries=self.n, mean_overlap=self.mean_overlap,
                    min_overlap=float(np.min(self.overlaps)) if self.overlaps else 1.0,
                    page_sets_differ=self.page_diff, max_abs=self.max_abs, rel_l2=self.rel_l2, lse_abs=self.lse_abs)

    def assert_ok(self, tol):
        s = self.summary()
        assert s["mean_overlap"] >= MIN_OVERLAP, s
        assert s["min_overlap"] >= MIN_OVERLAP_ANY, s
        if self.n_pages:
            assert self.page_diff <= max(1, int(MAX_PAGE_DIFF_SHARE * self.n_pages)), s
        assert s["max_abs"] <= tol["max_abs"] and s["rel_l2"] <= tol["rel_l2"], s
        assert s["lse_abs"] <= 1e-3, s


def check_invariants(cfg, t, sparse, n_sp):
    """Properties every selected set must have, whatever the scores."""
    sp = sparse[:n_sp]
    assert (sparse[n_sp:] == -1).all()
    if n_sp:
        assert (np.diff(sp) > 0).all() and sp[0] >= cfg.S and sp[-1] <= t - cfg.W


def check_prefill(wl, queries, check_attention=True, pages=None) -> Metrics:
    """wl: PrefillWorkload that has run (sparse_idx / out filled).  queries: absolute positions."""
    cfg = wl.cfg
    caches = ref.HostCaches(to_np(wl.keys["k"]), to_np(wl.keys["scale"]) if "scale" in wl.keys else None,
                            [to_np(k) for k in wl.k], [to_np(v) for v in wl.v], cfg.B, n_key=wl.n_key)
    m = Metrics()
    kw = dict(P=cfg.P, B=cfg.B, M=cfg.M, Ksp=cfg.Ksp, S=cfg.S, W=cfg.W)
    for t in queries:
        i = t - wl.q_pos0
        n_sp = int(wl.n_sparse[i])
        gpu_sparse = to_np(wl.sparse_idx[i])
        check_invariants(cfg, t, gpu_sparse, n_sp)
        ref_sparse, ref_pages = ref.select_query(t, to_np(wl.q_idx[i]), to_np(wl.w[i]), caches, hi_enable=cfg.hi_enable,
                                                 pooling=cfg.pooling, **kw)
        assert n_sp == len(ref_sparse), (t, n_sp, len(ref_sparse))
        gp = None
        if pages is not None:
            gp = to_np(pages[i])
            gp = gp[gp >= 0]
        m.add_select(gpu_sparse[:n_sp], ref_sparse, gp, ref_pages if gp is not None else None)
        if check_attention:
            outs, lses = ref.attend_query(t, [to_np(q[i]) for q in wl.q], caches, gpu_sparse[:n_sp], S=cfg.S, W=cfg.W,
                                          sm_scale=cfg.sm_scale, d_v=cfg.d_v)
            for r in range(cfg.R):
                m.add_out(to_np(wl.out[r][i]), outs[r], to_np(wl.lse[r][i]) if wl.lse[r] is not None else None, lses[r])
    return m


def decode_caches(wl, b, pools=None):
    """Logical caches of sequence b of a DecodeWorkload: (HostCaches, query position)."""
    cfg = wl.cfg
    if pools is None:
        pools = (to_np(wl.ctx_len), to_np(wl.page_table), to_np(wl.keys["k"]),
                 to_np(wl.keys["scale"]) if "scale" in wl.keys else None)
    ctx, table, k_pool, s_pool = pools
    n = int(ctx[b])
    # gather this sequence's K/V rows on the tensors' device (plumbing), widen on the host
    rows = torch.from_numpy(orc.paged_rows(np.arange(n), table[b], cfg.kv_page)).to(wl.k[0].device)
    k_l = [to_np(k[rows]) for k in wl.k]
    caches = ref.HostCaches(k_pool, s_pool, [], [], cfg.B, n_key=n, page_table_row=table[b], kv_page=cfg.kv_page)
    caches.k = k_l
    caches.v = [k[:, :cfg.d_v] for k in k_l] if cfg.mla else [to_np(v[rows]) for v in wl.v]
    return caches, n - 1


def check_decode(wl, seqs, check_attention=True) -> Metrics:
    cfg = wl.cfg
    m = Metrics()
    kw = dict(P=cfg.P, B=cfg.B, M=cfg.M, Ksp=cfg.Ksp, S=cfg.S, W=cfg.W)
    pools = (to_np(wl.ctx_len), to_np(wl.page_table), to_np(wl.keys["k"]),
             to_np(wl.keys["scale"]) if "scale" in wl.keys else None)
    for b in seqs:
        caches, t = decode_caches(wl, b, pools)
        n_sp = int(wl.n_sparse[b])
        gpu_sparse = to_np(wl.sparse_idx[b])
        check_invariants(cfg, t, gpu_sparse, n_sp)
        ref_sparse, _ = ref.select_query(t, to_np(wl.q_idx[b]), to_np(wl.w[b]), caches, hi_enable=cfg.hi_enable, **kw)
        assert n_sp == len(ref_sparse)
        m.add_select(gpu_sparse[:n_sp], ref_sparse)
        if check_attention:
            outs, lses = ref.attend_query(t, [to_np(q[b]) for q in wl.q], caches, gpu_sparse[:n_sp], S=cfg.S, W=cfg.W,
                                          sm_scale=cfg.sm_scale, d_v=cfg.d_v)
            for r in range(cfg.R):
                m.add_out(to_np(wl.out[r][b]), outs[r], to_np(wl.lse[r][b]) if wl.lse[r] is not None else None, lses[r])
    return m
