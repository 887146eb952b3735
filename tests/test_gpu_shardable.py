"""The shardable pieces (needs a B200): two-branch attention merged by LSE, and top-K re-ranked from shards.

Both are equivalences the paper states: the hybrid operator's sparse branch and sink+window branch merged by
online-softmax rescaling equal one softmax (Sec. 4.1.1); local top-K per cache shard followed by a re-rank of the
K*N candidates equals the global top-K (App. B).
"""
import numpy as np
import pytest
import torch

from oracle import lsa_oracle as orc
from paper_2608_01662_b200 import binding
from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import PrefillWorkload

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg1", "mla"])
def test_two_branches_merged_by_lse_equal_the_joint_softmax(cuda_device, name):
    cfg = CONFIGS["cfg1"] if name == "cfg1" else CONFIGS["cfg2"].replace(name="mla_br", L=3000, M=16, Ksp=512, W=256, R=1, seed=31)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()                                           # joint: out[0], lse[0]
    n = cfg.L
    new = lambda *shape, dt=torch.bfloat16: torch.empty(shape, dtype=dt, device=cuda_device)
    o_sp, l_sp = new(n, cfg.H, cfg.d_v), new(n, cfg.H, dt=torch.float32)
    o_fx, l_fx = new(n, cfg.H, cfg.d_v), new(n, cfg.H, dt=torch.float32)
    p_sparse = binding.make_params(cfg.replace(S=0, W=0))       # sparse branch only
    p_fixed = binding.make_params(cfg.replace(Ksp=0))           # sink + window branch only
    zeros = torch.zeros_like(wl.n_sparse)
    wl.ctx.sparse_attn(wl.q[0], wl.k[0], wl.v[0], wl.sparse_idx, wl.n_sparse, 0, n, n, o_sp, l_sp, params=p_sparse)
    wl.ctx.sparse_attn(wl.q[0], wl.k[0], wl.v[0], wl.sparse_idx, zeros, 0, n, n, o_fx, l_fx, params=p_fixed)
    o_m, l_m = new(n, cfg.H, cfg.d_v), new(n, cfg.H, dt=torch.float32)
    wl.ctx.merge([o_sp, o_fx], [l_sp, l_fx], n, o_m, l_m)
    assert wl.ctx.status() == 0
    # early queries have no sparse part: that branch reports an empty result
    assert torch.isinf(l_sp[0]).all() and (l_sp[0] < 0).all() and (o_sp[0] == 0).all()
    joint, merged = wl.out[0].float(), o_m.float()
    assert (joint - merged).abs().max() <= 2e-2
    assert (joint - merged).norm() / joint.norm() <= 5e-3
    assert (wl.lse[0] - l_m).abs().max() <= 1e-3
    # and the merge itself against the oracle's formula on the same parts (a sample of queries)
    for t in (0, cfg.S + cfg.W + 5, n // 2, n - 1):
        parts_o = [pu.to_np(o_sp[t]).astype(np.float64), pu.to_np(o_fx[t]).astype(np.float64)]
        parts_l = [pu.to_np(l_sp[t]).astype(np.float64), pu.to_np(l_fx[t]).astype(np.float64)]
        keep = [i for i in range(2) if np.isfinite(parts_l[i]).all()]
        want_o, want_l = orc.merge_partials([parts_o[i] for i in keep], [parts_l[i] for i in keep])
        assert np.abs(pu.to_np(o_m[t]) - want_o).max() <= 8e-3      # one bf16 rounding of values up to ~1
        assert np.abs(pu.to_np(l_m[t]) - want_l).max() <= 1e-4


def test_top_k_reranked_from_page_shards_equals_global(cuda_device):
    rng = np.random.default_rng(7)
    n_query, n_cand, K, page, n_shards = 8, 6000, 256, 64, 4
    scores = torch.from_numpy(np.round(rng.standard_normal((n_query, n_cand)), 2).astype(np.float32)).to(cuda_device)
    params = binding.make_params(CONFIGS["cfg1"].replace(S=0, W=0))
    ctx = binding.Context(params, n_query, n_cand, device=cuda_device)
    idx_g = torch.empty((n_query, K), dtype=torch.int32, device=cuda_device)
    cnt = torch.empty((n_query,), dtype=torch.int32, device=cuda_device)
    ctx.select(scores, None, 0, K, False, idx_g, cnt)                      # global top-K
    pos_all = torch.arange(n_cand, device=cuda_device, dtype=torch.int32)
    cands = []
    for r in range(n_shards):                                              # page i lives on rank i mod N
        mine = pos_all[(pos_all // page) % n_shards == r]
        sc = scores[:, mine.long()].contiguous()
        pos = mine[None].expand(n_query, -1).contiguous()
        idx_l = torch.empty((n_query, K), dtype=torch.int32, device=cuda_device)
        ctx.select(sc, pos, 0, K, False, idx_l, cnt)                       # local top-K of the shard
        cands.append(idx_l)
    cand = torch.sort(torch.cat(cands, dim=1), dim=1).values               # K*N candidates, ascending positions
    cand_sc = torch.gather(scores, 1, cand.long())
    idx_r = torch.empty((n_query, K), dtype=torch.int32, device=cuda_device)
    ctx.select(cand_sc, cand, 0, K, False, idx_r, cnt)                     # re-rank
    assert ctx.status() == 0
    assert torch.equal(idx_r, idx_g)
