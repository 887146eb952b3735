"""Seeded synthetic inputs, shared by the CUDA path's callers and by the oracle's tests.

This module holds none of the method's arithmetic: it only draws random
tensors with the shapes and laws of the workloads and stores them in the
formats the caches use (bf16, or e4m3 codes with a per-token fp32 scale).
Every per-row tensor is drawn in chunks of GEN_ROWS rows, each chunk from its
own seed, so that any row range of a huge tensor can be regenerated alone.

Laws: indexer q_I, k_I ~ N(0, 1/d_I); head weights w ~ N(0, 1/H_I); attention
q, k, v (or the MLA latent) ~ N(0, 1).  With boost_prob > 0 a Bernoulli share of
tokens has its indexer key multiplied by boost_gain before it is stored.  With
segment_corr = rho > 0 the indexer keys of each run of segment_len consecutive
tokens share a direction: k_s = sqrt(rho) c_seg + sqrt(1 - rho) e_s with c, e
of the same law (text whose neighbouring tokens attend alike, the structure a
page-level score can see); the marginal law of a key is unchanged.
"""
from __future__ import annotations

import math

import torch

from .configs import LsaConfig

GEN_ROWS = 16384

T_QI, T_KI, T_W, T_BOOST, T_SEG, T_Q, T_KV, T_V, T_CTX, T_PERM = 0, 1, 2, 3, 4, 10, 20, 40, 30, 31

E4M3_MAX = 448.0


def _generator(cfg: LsaConfig, tensor_id: int, chunk_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + tensor_id * 1009 + chunk_id)
    return g


def _rows(cfg, tensor_id, row0, nrows, row_shape, std, device, uniform=False):
    """Rows [row0, row0+nrows) of the tensor `tensor_id`, fp32, shape [nrows, *row_shape]."""
    out = torch.empty((nrows, *row_shape), dtype=torch.float32, device=device)
    c0, c1 = row0 // GEN_ROWS, (row0 + nrows - 1) // GEN_ROWS if nrows > 0 else -1
    for c in range(c0, c1 + 1):
        g = _generator(cfg, tensor_id, c, device)
        if uniform:
            chunk = torch.rand((GEN_ROWS, *row_shape), generator=g, device=device, dtype=torch.float32)
        else:
            chunk = torch.randn((GEN_ROWS, *row_shape), generator=g, device=device, dtype=torch.float32)
            chunk *= std
        a = max(row0, c * GEN_ROWS)
        b = min(row0 + nrows, (c + 1) * GEN_ROWS)
        out[a - row0:b - row0] = chunk[a - c * GEN_ROWS:b - c * GEN_ROWS]
        del chunk
    return out


def indexer_queries(cfg: LsaConfig, row0: int, nrows: int, device):
    """(q_I bf16 [n, H_I, d_I], w fp32 [n, H_I]) for query rows row0..row0+nrows."""
    q = _rows(cfg, T_QI, row0, nrows, (cfg.H_I, cfg.d_I), 1.0 / math.sqrt(cfg.d_I), device)
    w = _rows(cfg, T_W, row0, nrows, (cfg.H_I,), 1.0 / math.sqrt(cfg.H_I), device)
    return q.to(torch.bfloat16), w


def quantize_e4m3(k: torch.Tensor):
    """fp32 rows -> (uint8 e4m3 codes, fp32 per-row scale = amax/448, 1 when the row is zero)."""
    amax = k.abs().amax(dim=-1)
    scale = torch.where(amax > 0, amax / E4M3_MAX, torch.ones_like(amax))
    codes = (k / scale[..., None]).clamp_(-E4M3_MAX, E4M3_MAX).to(torch.float8_e4m3fn).view(torch.uint8)
    return codes, scale


def indexer_keys(cfg: LsaConfig, n_rows: int, device):
    """Indexer key cache rows 0..n_rows: {"k": bf16 [n, d_I]} or {"k": uint8 codes, "scale": fp32 [n]}."""
    ks, scales = [], []
    for r0 in range(0, n_rows, GEN_ROWS):
        n = min(GEN_ROWS, n_rows - r0)
        k = _rows(cfg, T_KI, r0, n, (cfg.d_I,), 1.0 / math.sqrt(cfg.d_I), device)
        if cfg.segment_corr > 0:
            seg0, seg1 = r0 // cfg.segment_len, (r0 + n - 1) // cfg.segment_len
            c = _rows(cfg, T_SEG, seg0, seg1 - seg0 + 1, (cfg.d_I,), 1.0 / math.sqrt(cfg.d_I), device)
            seg_of = torch.arange(r0, r0 + n, device=device) // cfg.segment_len - seg0
            k = math.sqrt(cfg.segment_corr) * c[seg_of] + math.sqrt(1.0 - cfg.segment_corr) * k
        if cfg.boost_prob > 0:
            u = _rows(cfg, T_BOOST, r0, n, (), 1.0, device, uniform=True)
            k = torch.where((u < cfg.boost_prob)[:, None], k * cfg.boost_gain, k)
        if cfg.key_dtype == "e4m3":
            c, s = quantize_e4m3(k)
            ks.append(c)
            scales.append(s)
        else:
            ks.append(k.to(torch.bfloat16))
    out = {"k": torch.cat(ks) if ks else torch.empty((0, cfg.d_I), device=device)}
    if cfg.key_dtype == "e4m3":
        out["scale"] = torch.cat(scales)
    return out


def attn_queries(cfg: LsaConfig, r: int, row0: int, nrows: int, device):
    """q of layer r, bf16 [n, H, d_qk]."""
    return _rows(cfg, T_Q + r, row0, nrows, (cfg.H, cfg.d_qk), 1.0, device).to(torch.bfloat16)


def attn_kv(cfg: LsaConfig, r: int, n_rows: int, device):
    """(k, v) of layer r.  MLA: k is the latent [n, d_qk] and v is the view k[:, :d_v]."""
    def rows(tid, d):
        parts = [_rows(cfg, tid, r0, min(GEN_ROWS, n_rows - r0), (d,), 1.0, device).to(torch.bfloat16)
                 for r0 in range(0, n_rows, GEN_ROWS)]
        return torch.cat(parts) if parts else torch.empty((0, d), dtype=torch.bfloat16, device=device)
    k = rows(T_KV + r, cfg.d_qk)
    if cfg.mla:
        return k, k[:, :cfg.d_v]
    return k, rows(T_V + r, cfg.d_v)


def decode_layout(cfg: LsaConfig, device):
    """(ctx_len int32 [batch], page_table int32 [batch, max_pages], n_phys_pages).

    Context lengths are uniform integers in [ctx_lo, ctx_hi]; the physical pages
    are a random permutation dealt to the sequences in order (enough of them
    for cfg.ctx_grow more tokens per sequence); unused table entries are -1.
    """
    g = _generator(cfg, T_CTX, 0, "cpu")
    ctx = torch.randint(cfg.ctx_lo, cfg.ctx_hi + 1, (cfg.batch,), generator=g, dtype=torch.int64)
    n_pages = (ctx + cfg.ctx_grow + cfg.kv_page - 1) // cfg.kv_page   # room for ctx_grow appended tokens
    n_pg = int(n_pages.sum())
    perm = torch.randperm(n_pg, generator=_generator(cfg, T_PERM, 0, "cpu"))
    table = torch.full((cfg.batch, int(n_pages.max())), -1, dtype=torch.int32)
    off = 0
    for b in range(cfg.batch):
        n = int(n_pages[b])
        table[b, :n] = perm[off:off + n].to(torch.int32)
        off += n
    return ctx.to(torch.int32).to(device), table.to(device), n_pg
