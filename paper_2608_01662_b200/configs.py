"""Workload descriptions: the five synthetic configurations and small test variants.

Pure data.  Symbols follow the paper: P page size, B sub-block size, M recalled
pages (Sec. 3.3), S/W/Ksp = K_sink / K_swa / K_sparse (Eq. 6), R = cross-layer
group size N (Sec. 3.2), H_I/d_I indexer heads and head dim (Eq. 1).
"""
from __future__ import annotations

import dataclasses
import math


@dataclasses.dataclass(frozen=True)
class LsaConfig:
    name: str
    seed: int
    mode: str            # "prefill" | "decode"
    L: int               # prefill: sequence length; decode: unused (see ctx_lo/ctx_hi)
    H_I: int
    d_I: int
    key_dtype: str       # "bf16" | "e4m3"
    P: int
    B: int
    M: int
    Ksp: int
    S: int
    W: int
    H: int
    d_qk: int
    d_v: int
    mla: bool            # True: one latent row is key (d_qk dims) and value (first d_v dims)
    sm_scale: float
    R: int
    q_chunk: int = 0     # 0 = whole sequence at once
    batch: int = 1
    ctx_lo: int = 0      # decode: context length ~ U{ctx_lo..ctx_hi}
    ctx_hi: int = 0
    kv_page: int = 0     # decode: tokens per physical cache page
    ctx_grow: int = 0    # decode: tokens each sequence can still append (pages mapped ahead)
    boost_prob: float = 0.0   # share of tokens whose indexer key is scaled by boost_gain
    boost_gain: float = 1.0
    segment_corr: float = 0.0  # share of an indexer key's variance that is common to its run of segment_len tokens
    segment_len: int = 64
    hi_enable: bool = True
    pooling: str = "mean"   # coarse-stage pooling: "mean" (Eq. 9) or "minmax" (Eq. 13)

    def replace(self, **kw) -> "LsaConfig":
        return dataclasses.replace(self, **kw)


_MLA = dict(H=64, d_qk=576, d_v=512, mla=True, sm_scale=1.0 / math.sqrt(576.0))

CONFIGS = {
    "cfg1": LsaConfig("cfg1", 0, "prefill", 2048, 8, 64, "bf16", 64, 8, 8, 256, 4, 128,
                      16, 128, 128, False, 1.0 / math.sqrt(128.0), 1),
    "cfg2": LsaConfig("cfg2", 1, "prefill", 32768, 64, 128, "bf16", 64, 8, 64, 2048, 4, 512,
                      R=2, **_MLA),
    "cfg3": LsaConfig("cfg3", 2, "prefill", 131072, 64, 128, "e4m3", 128, 8, 32, 2048, 4, 1024,
                      R=4, boost_prob=0.05, boost_gain=4.0, **_MLA),
    "cfg4": LsaConfig("cfg4", 3, "decode", 0, 64, 128, "e4m3", 64, 8, 64, 2048, 4, 256,
                      R=4, batch=64, ctx_lo=16384, ctx_hi=131072, kv_page=64, **_MLA),
    # cfg3 cut to 16K tokens and one layer: small enough for multi-pass ncu captures, still larger than L2
    "cfg3_16k": LsaConfig("cfg3_16k", 2, "prefill", 16384, 64, 128, "e4m3", 128, 8, 32, 2048, 4, 1024,
                          R=1, boost_prob=0.05, boost_gain=4.0, **_MLA),
    "cfg5": LsaConfig("cfg5", 4, "prefill", 1048576, 64, 128, "e4m3", 256, 8, 16, 2048, 4, 2048,
                      R=4, q_chunk=16384, **_MLA),
}
