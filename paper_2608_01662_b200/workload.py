"""Device-resident synthetic workloads driven through the C ABI (used by the tests, smoke and bench)."""
from __future__ import annotations

import torch

from . import binding, inputs
from .configs import LsaConfig


class PrefillWorkload:
    """One sequence of cfg.L tokens (or the query range [q_pos0, q_pos0 + n_query) of it).

    The caches (indexer keys, mean keys, per-layer K/V) cover positions [0, n_key); the per-query
    tensors cover the query range only.
    """

    def __init__(self, cfg: LsaConfig, device="cuda:0", q_pos0: int = 0, n_query: int | None = None,
                 n_key: int | None = None, with_lse: bool = True, make_ctx: bool = True):
        assert cfg.mode == "prefill"
        self.cfg, self.device = cfg, torch.device(device)
        self.q_pos0 = q_pos0
        self.n_query = cfg.L - q_pos0 if n_query is None else n_query
        self.n_key = cfg.L if n_key is None else n_key
        dev = self.device
        self.params = binding.make_params(cfg)
        self.keys = inputs.indexer_keys(cfg, self.n_key, dev)
        self.q_idx, self.w = inputs.indexer_queries(cfg, q_pos0, self.n_query, dev)
        self.k, self.v, self.q, self.out, self.lse = [], [], [], [], []
        for r in range(cfg.R):
            k, v = inputs.attn_kv(cfg, r, self.n_key, dev)
            self.k.append(k)
            self.v.append(v)
            self.q.append(inputs.attn_queries(cfg, r, q_pos0, self.n_query, dev))
            self.out.append(torch.empty((self.n_query, cfg.H, cfg.d_v), dtype=torch.bfloat16, device=dev))
            self.lse.append(torch.empty((self.n_query, cfg.H), dtype=torch.float32, device=dev) if with_lse else None)
        n_sub = (self.n_key + cfg.B - 1) // cfg.B
        # mean keys, or [k_max | k_min] rows for the MinMax pooling variant
        self.kmean = torch.empty((n_sub, cfg.d_I * (2 if cfg.pooling == "minmax" else 1)), dtype=torch.bfloat16, device=dev)
        self.sparse_idx = torch.empty((self.n_query, cfg.Ksp), dtype=torch.int32, device=dev)
        self.n_sparse = torch.empty((self.n_query,), dtype=torch.int32, device=dev)
        self.ctx = binding.Context(self.params, self.n_query, self.n_key, 1, device=dev) if make_ctx else None

    def prepare(self):
        """Cache maintenance that happens once per sequence, not per group: the mean-key cache."""
        self.ctx.block_means(self.keys["k"], self.keys.get("scale"), self.n_key, self.kmean)

    def index(self, pages_out=None):
        self.ctx.index(self.q_idx, self.w, self.keys["k"], self.keys.get("scale"), self.kmean, self.q_pos0,
                       self.n_query, self.n_key, self.sparse_idx, self.n_sparse, pages_out)

    def attend(self, r: int):
        self.ctx.sparse_attn(self.q[r], self.k[r], self.v[r], self.sparse_idx, self.n_sparse, self.q_pos0,
                             self.n_query, self.n_key, self.out[r], self.lse[r])

    def step(self):
        """One pass of the whole hot path over the batch: a1..a7."""
        self.ctx.layer_group(self.q_idx, self.w, self.keys["k"], self.keys.get("scale"), self.kmean, self.q_pos0,
                             self.n_query, self.n_key, self.q, self.k, self.v, self.out,
                             self.lse if self.lse[0] is not None else None, self.sparse_idx, self.n_sparse)

    def units(self) -> int:
        return self.n_query


class DecodeWorkload:
    """cfg.batch sequences with paged caches and one new query token each."""

    def __init__(self, cfg: LsaConfig, device="cuda:0", with_lse: bool = True, make_ctx: bool = True):
        assert cfg.mode == "decode"
        self.cfg, self.device = cfg, torch.device(device)
        dev = self.device
        self.params = binding.make_params(cfg)
        self.ctx_len, self.page_table, self.n_pg = inputs.decode_layout(cfg, dev)
        n_rows = self.n_pg * cfg.kv_page
        self.keys = inputs.indexer_keys(cfg, n_rows, dev)
        self.q_idx, self.w = inputs.indexer_queries(cfg, 0, cfg.batch, dev)
        self.k, self.v, self.q, self.out, self.lse = [], [], [], [], []
        for r in range(cfg.R):
            k, v = inputs.attn_kv(cfg, r, n_rows, dev)
            self.k.append(k)
            self.v.append(v)
            self.q.append(inputs.attn_queries(cfg, r, 0, cfg.batch, dev))
            self.out.append(torch.empty((cfg.batch, cfg.H, cfg.d_v), dtype=torch.bfloat16, device=dev))
            self.lse.append(torch.empty((cfg.batch, cfg.H), dtype=torch.float32, device=dev) if with_lse else None)
        self.kmean = torch.zeros((n_rows // cfg.B, cfg.d_I), dtype=torch.bfloat16, device=dev)
        self.sparse_idx = torch.empty((cfg.batch, cfg.Ksp), dtype=torch.int32, device=dev)
        self.n_sparse = torch.empty((cfg.batch,), dtype=torch.int32, device=dev)
        max_ctx = self.page_table.shape[1] * cfg.kv_page
        self.ctx = binding.Context(self.params, cfg.batch, max_ctx, cfg.batch, device=dev) if make_ctx else None

    def prepare(self):
        self.ctx.block_means(self.keys["k"], self.keys.get("scale"), 0, self.kmean, self.page_table, self.ctx_len)

    def index(self, pages_out=None):
        self.ctx.index(self.q_idx, self.w, self.keys["k"], self.keys.get("scale"), self.kmean, 0, self.cfg.batch, 0,
                       self.sparse_idx, self.n_sparse, pages_out, self.page_table, self.ctx_len)

    def step(self):
        self.ctx.layer_group(self.q_idx, self.w, self.keys["k"], self.keys.get("scale"), self.kmean, 0,
                             self.cfg.batch, 0, self.q, self.k, self.v, self.out,
                             self.lse if self.lse[0] is not None else None, self.sparse_idx, self.n_sparse,
                             self.page_table, self.ctx_len)

    def units(self) -> int:
        return self.cfg.batch


def make_workload(cfg: LsaConfig, device="cuda:0", **kw):
    return DecodeWorkload(cfg, device, **kw) if cfg.mode == "decode" else PrefillWorkload(cfg, device, **kw)
