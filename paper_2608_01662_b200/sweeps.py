"""Recall-versus-cost sweep of the coarse stage: pooling method, sub-block size B and recall budget M.

    python -m paper_2608_01662_b200.sweeps [--seq-len 32768] [--q-tail 2048] [--boost 0.02,4]

For every setting the last `q_tail` queries of a synthetic length-L prefill are indexed twice on the GPU: with the
two-stage selection (Eq. 9-12, mean pooling or the MinMax pooling of Eq. 13) and with the flat selection of Eq. 7
(`hi_enable = 0`), which is what the hierarchy approximates.  Reported per setting:

    recall   mean over queries of |S_hier & S_flat| / |S_flat|   (the Overlap of App. C on the sparse part)
    ms       device time of the coarse stage and of the fine stage + selections (CUDA-event pairs of the library)

Everything is computed by the CUDA library; no oracle is involved.  The inputs follow the package's seeded recipe
(Gaussian keys and queries; `--segment-corr rho` gives the keys of each run of 64 tokens a common direction, the
locality a page-level score relies on; `--boost p,g` multiplies a share p of the keys by g so that a few tokens
stand out of their neighbourhood, the regime in which the pooling method matters).
"""
from __future__ import annotations

import argparse
import json

import torch

from .configs import CONFIGS
from .workload import DecodeWorkload, PrefillWorkload


def _index(cfg, dev, q_pos0, n_query, steps=3):
    wl = PrefillWorkload(cfg.replace(R=0), dev, q_pos0=q_pos0, n_query=n_query, with_lse=False)
    wl.prepare()
    wl.index()
    wl.ctx.profile_enable(True)
    for _ in range(steps):
        wl.index()
    prof = wl.ctx.profile_read()
    wl.ctx.profile_enable(False)
    assert wl.ctx.status() == 0
    ms = {k: v[0] / steps for k, v in prof.items() if v[1] > 0}
    return wl.sparse_idx.clone(), wl.n_sparse.clone(), ms


def _recall(idx_a, n_a, idx_ref, n_ref):
    """Mean over rows of |a & ref| / |ref| for ascending, -1 padded index lists (rows with empty ref count as 1)."""
    k = idx_ref.shape[1]
    big = torch.iinfo(torch.int32).max
    a = torch.where(idx_a >= 0, idx_a, torch.full_like(idx_a, big - 1))
    r = torch.where(idx_ref >= 0, idx_ref, torch.full_like(idx_ref, big))
    pos = torch.searchsorted(a.contiguous(), r.contiguous()).clamp_(max=k - 1)
    hit = (torch.gather(a, 1, pos) == r) & (idx_ref >= 0)
    n = n_ref.clamp(min=1).to(torch.float32)
    rec = torch.where(n_ref > 0, hit.sum(dim=1).to(torch.float32) / n, torch.ones_like(n))
    return float(rec.mean())


def decode_table(dev, batch=4, steps=20):
    """Decode cost against context length (the counterpart of the paper's Table 1): `batch` sequences of equal length,
    one query token each, one attention layer; indexer kernels and the attention kernel timed by the library's event
    pairs, for the hierarchical indexer and for the flat one (hi_enable = 0)."""
    for ctx in (4096, 16384, 65536, 262144, 1048576):
        for flat in (False, True):
            cfg = CONFIGS["cfg4"].replace(name="decode_table", batch=batch, ctx_lo=ctx, ctx_hi=ctx, R=1, hi_enable=not flat)
            wl = DecodeWorkload(cfg, dev, with_lse=False)
            wl.prepare()
            for _ in range(3):
                wl.step()
            wl.ctx.profile_enable(True)
            for _ in range(steps):
                wl.step()
            prof = wl.ctx.profile_read()
            wl.ctx.profile_enable(False)
            assert wl.ctx.status() == 0
            us = {k: round(v[0] / steps * 1e3, 1) for k, v in prof.items() if v[1] > 0}
            indexer = round(sum(v for k, v in us.items() if k != "sparse_attn"), 1)
            print(json.dumps(dict(context=ctx, batch=batch, indexer="flat" if flat else "hierarchical", kernels_us=us,
                                  indexer_us=indexer, attention_us=us.get("sparse_attn", 0.0))), flush=True)
            del wl
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--decode-table", action="store_true",
                    help="decode indexer and attention time against context length, hierarchical and flat, instead of the sweep")
    ap.add_argument("--seq-len", type=int, default=32768)
    ap.add_argument("--q-tail", type=int, default=2048)
    ap.add_argument("--boost", default="0.02,4", help="share of boosted keys and their gain; '0,1' = none")
    ap.add_argument("--segment-corr", type=float, default=0.5,
                    help="share of a key's variance common to its run of 64 tokens; 0 = independent keys")
    ap.add_argument("--device", default="cuda:0")
    args = ap.parse_args()
    dev = torch.device(args.device)
    if args.decode_table:
        decode_table(dev)
        return
    bp, bg = (float(x) for x in args.boost.split(","))
    base = CONFIGS["cfg3"].replace(name="sweep", L=args.seq_len, boost_prob=bp, boost_gain=bg,
                                   segment_corr=args.segment_corr)
    q0 = args.seq_len - args.q_tail
    flat_idx, flat_n, flat_ms = _index(base.replace(hi_enable=False), dev, q0, args.q_tail)
    rows = []
    for P, B in ((128, 4), (128, 8), (128, 16), (256, 32)):
        for M_tokens in (2048, 4096):
            M = M_tokens // P
            for pooling in ("mean", "minmax"):
                cfg = base.replace(P=P, B=B, M=M, pooling=pooling)
                idx, n, ms = _index(cfg, dev, q0, args.q_tail)
                rows.append(dict(pooling=pooling, P=P, B=B, M=M, budget_tokens=M * P,
                                 recall=_recall(idx, n, flat_idx, flat_n),
                                 coarse_ms=ms.get("coarse_score", 0.0), fine_ms=ms.get("fine_select", 0.0)))
                print(json.dumps(rows[-1]), flush=True)
    print(json.dumps({"flat_ms": flat_ms, "seq_len": args.seq_len, "q_tail": args.q_tail, "boost": [bp, bg],
                      "segment_corr": args.segment_corr}))


if __name__ == "__main__":
    main()
