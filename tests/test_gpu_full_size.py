"""Parity at the benchmark's sizes and launch configuration, on sampled queries (needs a B200)."""
import pytest
import torch

from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import DecodeWorkload, PrefillWorkload

import parity_util as pu

pytestmark = pytest.mark.gpu


def _free():
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def test_cfg2_prefill_32k_sampled(cuda_device):
    cfg = CONFIGS["cfg2"]
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 200, seed=2))
    print("cfg2", m.summary())
    m.assert_ok(pu.TOL_BF16)
    del wl
    _free()


def test_cfg3_prefill_128k_sampled(cuda_device):
    """The configuration bench.py times: L = 131072, fp8 indexer keys, R = 4, one lsa_layer_group call."""
    cfg = CONFIGS["cfg3"]
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 200, seed=3))
    print("cfg3", m.summary())
    m.assert_ok(pu.TOL_FP8)
    # properties that hold for every query at full size
    n_sp = wl.n_sparse.to(torch.int64)
    t = torch.arange(cfg.L, device=cuda_device)
    assert torch.equal(n_sp, (t - cfg.W - cfg.S + 1).clamp(0, cfg.Ksp))
    idx = wl.sparse_idx.to(torch.int64)
    valid = idx >= 0
    assert torch.equal(valid.sum(1), n_sp)
    assert ((idx <= (t - cfg.W)[:, None]) | ~valid).all() and ((idx >= cfg.S) | ~valid).all()
    assert ((idx[:, 1:] > idx[:, :-1]) | ~valid[:, 1:]).all()
    for r in range(cfg.R):
        assert torch.isfinite(wl.out[r].float()).all()
    del wl
    _free()


def test_cfg4_decode_all_sequences(cuda_device):
    cfg = CONFIGS["cfg4"]
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print("cfg4", m.summary())
    m.assert_ok(pu.TOL_FP8)
    del wl
    _free()


@pytest.mark.parametrize("chunk", [0, 1, 17, 37, 50, 63])
def test_cfg5_prefill_1m_chunks(cuda_device, chunk):
    """1M-token caches resident; the queries of one 16384-query chunk at a time.  Six chunks (the first, where the
    number of eligible pages crosses M, its neighbour, four spread over the rest including the last) with the boundary
    positions plus 34 random queries each: more than 200 random queries in total."""
    cfg = CONFIGS["cfg5"]
    wl = PrefillWorkload(cfg, cuda_device, q_pos0=chunk * cfg.q_chunk, n_query=cfg.q_chunk)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, wl.q_pos0, wl.n_query, 34, seed=chunk))
    print("cfg5 chunk", chunk, m.summary())
    m.assert_ok(pu.TOL_FP8)
    del wl
    _free()
