"""Runs the oracle on host copies of a workload's tensors (test infrastructure only).

Takes numpy arrays and plain numbers; knows nothing of the CUDA library.  bf16 tensors must be
widened to float32/float64 by the caller (exactly), e4m3 keys come as uint8 codes plus scales.
"""
from __future__ import annotations

import numpy as np

from . import lsa_oracle as orc


class HostCaches:
    """Logical (unpaged) view of one sequence's caches, in float64."""

    def __init__(self, k_idx, k_scale, k_layers, v_layers, B, n_key=None, page_table_row=None, kv_page=None):
        def logical(pool):
            pool = np.asarray(pool)
            if page_table_row is None:
                return pool[:n_key] if n_key is not None else pool
            return orc.gather_paged(pool, page_table_row, n_key, kv_page)
        k_idx = logical(k_idx)
        if k_scale is not None:
            self.k_hat = orc.dequant_keys(k_idx, logical(k_scale))
        else:
            self.k_hat = k_idx.astype(np.float64)
        self.km = orc.block_means(self.k_hat, B)
        self.B = B
        self._minmax = None
        self.k = [logical(k).astype(np.float64) for k in k_layers]
        self.v = [logical(v).astype(np.float64) for v in v_layers]


    def minmax(self):
        """(k_max, k_min) caches of Eq. 13, built on first use."""
        if self._minmax is None:
            self._minmax = orc.block_minmax(self.k_hat, self.B)
        return self._minmax


def select_query(t, q_I, w, caches: HostCaches, *, P, B, M, Ksp, S, W, hi_enable=True, pooling="mean"):
    return orc.select_sparse(t, np.asarray(q_I, dtype=np.float64), np.asarray(w, dtype=np.float64), caches.k_hat,
                             caches.km, P=P, B=B, M=M, Ksp=Ksp, S=S, W=W, hi_enable=hi_enable,
                             minmax=caches.minmax() if pooling == "minmax" else None)


def attend_query(t, q_layers, caches: HostCaches, sparse, *, S, W, sm_scale, d_v):
    """Eq. 3 for every layer of the group on a given sparse set (e.g. the one the GPU selected)."""
    S_t = orc.index_set(t, S, W, sparse)
    outs, lses = [], []
    for r, q in enumerate(q_layers):
        o, l = orc.attend(np.asarray(q, dtype=np.float64), caches.k[r], caches.v[r][:, :d_v], S_t, sm_scale)
        outs.append(o)
        lses.append(l)
    return outs, lses


def overlap(gpu_sparse, ref_sparse):
    """card(S_gpu & S_ref) / card(S_ref)  (the Overlap of App. C on the sparse part); 1 when both are empty."""
    a, b = set(int(x) for x in gpu_sparse), set(int(x) for x in ref_sparse)
    if not b:
        return 1.0 if not a else 0.0
    return len(a & b) / len(b)
