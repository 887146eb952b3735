"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle (needs a B200)."""
import math

import numpy as np
import pytest
import torch

from oracle import lsa_oracle as orc
from paper_2608_01662_b200 import binding
from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import DecodeWorkload, PrefillWorkload

import parity_util as pu

pytestmark = pytest.mark.gpu

SMALL_MLA = CONFIGS["cfg2"].replace(name="mla_small", L=4096, M=16, Ksp=512, W=256, seed=11)
SMALL_FP8 = CONFIGS["cfg3"].replace(name="fp8_small", L=6000, M=8, Ksp=512, W=384, R=2, seed=12)
SMALL_DEC = CONFIGS["cfg4"].replace(name="dec_small", batch=6, ctx_lo=1500, ctx_hi=6000, M=16, Ksp=512, R=2, seed=13)


def _sel_params(S=0, W=0):
    return binding.make_params(CONFIGS["cfg1"].replace(S=S, W=W))


# ---------------------------------------------------------------- selection alone: bit exact
@pytest.mark.parametrize("n_cand,k", [(1, 1), (37, 8), (1000, 256), (4096, 2048), (5000, 5000), (70000, 2048), (300, 512),
                                      (20000, 5000), (333333, 2048)])
def test_select_is_bit_exact_on_given_scores(cuda_device, n_cand, k):
    g = torch.Generator(device="cpu").manual_seed(n_cand * 7 + k)
    n_query = 9
    scores = torch.randn(n_query, n_cand, generator=g)
    scores[:, ::5] = torch.round(scores[:, ::5] * 2) / 2          # many exact ties
    scores[1] = 0.0
    scores[2, ::2] = -0.0                                          # +0 / -0 are one value
    scores[3] = -scores[3].abs()
    params = _sel_params()
    ctx = binding.Context(params, n_query, n_cand, device=cuda_device)
    d_scores = scores.to(cuda_device)
    idx = torch.empty((n_query, k), dtype=torch.int32, device=cuda_device)
    cnt = torch.empty((n_query,), dtype=torch.int32, device=cuda_device)
    ctx.select(d_scores, None, 0, k, False, idx, cnt)
    assert ctx.status() == 0
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    for i in range(n_query):
        want = orc.select_fp32(scores[i].numpy(), None, 0, k, apply_range=False)
        assert cnt[i] == len(want)
        assert np.array_equal(idx[i, :cnt[i]], want) and (idx[i, cnt[i]:] == -1).all()


def test_select_with_positions_range_and_leading_dimension(cuda_device):
    rng = np.random.default_rng(5)
    n_query, n_cand, ld, k, S, W, q_pos0 = 16, 700, 768, 100, 4, 64, 500
    scores = torch.from_numpy(np.round(rng.standard_normal((n_query, ld)), 1).astype(np.float32))
    params = _sel_params(S, W)
    ctx = binding.Context(params, n_query, 4096, device=cuda_device)
    idx = torch.empty((n_query, k), dtype=torch.int32, device=cuda_device)
    cnt = torch.empty((n_query,), dtype=torch.int32, device=cuda_device)
    d_scores = scores.to(cuda_device)[:, :n_cand]                 # row stride 768, 700 columns
    ctx.select(d_scores, None, q_pos0, k, True, idx, cnt)
    for i in range(n_query):
        want = orc.select_fp32(scores[i, :n_cand].numpy(), None, q_pos0 + i, k, apply_range=True, S=S, W=W)
        assert np.array_equal(idx[i, :int(cnt[i])].cpu().numpy(), want)
    # explicit candidate positions with holes, ascending per row
    pos = np.stack([np.sort(rng.permutation(5000)[:n_cand]) for _ in range(n_query)]).astype(np.int32)
    pos[:, ::9] = -1
    d_pos = torch.from_numpy(pos).to(cuda_device)
    d_sc = scores[:, :n_cand].contiguous().to(cuda_device)
    ctx.select(d_sc, d_pos, 0, k, False, idx, cnt)
    for i in range(n_query):
        want = orc.select_fp32(scores[i, :n_cand].numpy(), pos[i], 0, k, apply_range=False)
        assert np.array_equal(idx[i, :int(cnt[i])].cpu().numpy(), want)
    assert ctx.status() == 0


def test_select_of_long_rows_with_positions_and_range(cuda_device):
    """Rows long enough for the cluster selection (eight blocks per row): the scoring range cuts the row, explicit
    candidate positions have holes, many scores tie, and a row has fewer candidates than k."""
    rng = np.random.default_rng(8)
    n_query, n_cand, k, S, W, q_pos0 = 5, 40000, 3000, 4, 300, 39000
    scores = torch.from_numpy(np.round(rng.standard_normal((n_query, n_cand)), 2).astype(np.float32))
    params = _sel_params(S, W)
    ctx = binding.Context(params, n_query, n_cand, device=cuda_device)
    idx = torch.empty((n_query, k), dtype=torch.int32, device=cuda_device)
    cnt = torch.empty((n_query,), dtype=torch.int32, device=cuda_device)
    d_sc = scores.to(cuda_device)
    ctx.select(d_sc, None, q_pos0, k, True, idx, cnt)              # columns are positions; query i sits at q_pos0 + i
    for i in range(n_query):
        want = orc.select_fp32(scores[i].numpy(), None, q_pos0 + i, k, apply_range=True, S=S, W=W)
        assert cnt[i] == len(want)
        assert np.array_equal(idx[i, :int(cnt[i])].cpu().numpy(), want)
    pos = np.stack([np.sort(rng.permutation(300000)[:n_cand]) for _ in range(n_query)]).astype(np.int32)
    pos[:, ::7] = -1
    pos[4, 2000:] = -1                                             # 2000 columns, of which 1714 are present: fewer than k
    d_pos = torch.from_numpy(pos).to(cuda_device)
    ctx.select(d_sc, d_pos, 0, k, False, idx, cnt)
    for i in range(n_query):
        want = orc.select_fp32(scores[i].numpy(), pos[i], 0, k, apply_range=False)
        assert cnt[i] == len(want)
        got = idx[i].cpu().numpy()
        assert np.array_equal(got[:len(want)], want) and (got[len(want):] == -1).all()
    assert ctx.status() == 0


# ---------------------------------------------------------------- mean cache
@pytest.mark.parametrize("cfg", [CONFIGS["cfg1"], SMALL_FP8], ids=lambda c: c.name)
def test_block_means_match_oracle(cuda_device, cfg):
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    k_hat = (orc.dequant_keys(pu.to_np(wl.keys["k"]), pu.to_np(wl.keys["scale"])) if "scale" in wl.keys
             else pu.to_np(wl.keys["k"]).astype(np.float64))
    want = orc.block_means(k_hat, cfg.B)
    got = pu.to_np(wl.kmean).astype(np.float64)
    assert got.shape == want.shape
    # fp32 accumulation then one rounding vs fp64 then one rounding: equal except rare 1-ulp ties
    diff = got != want
    assert diff.mean() < 2e-3
    assert np.abs(got - want).max() <= np.abs(want).max() * 2.0 ** -7


# ---------------------------------------------------------------- whole path, small shapes
def test_cfg1_every_query(cuda_device):
    cfg = CONFIGS["cfg1"]
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    pages = torch.empty((cfg.L, cfg.M), dtype=torch.int32, device=cuda_device)
    wl.index(pages)
    sparse_from_index = wl.sparse_idx.clone()
    wl.step()
    assert wl.ctx.status() == 0
    assert torch.equal(sparse_from_index, wl.sparse_idx)          # the group runs the same indexer
    m = pu.check_prefill(wl, range(cfg.L), pages=pages)
    print("cfg1", m.summary())
    m.assert_ok(pu.TOL_BF16)


@pytest.mark.parametrize("cfg", [SMALL_MLA, SMALL_FP8], ids=lambda c: c.name)
def test_small_mla_prefill(cuda_device, cfg):
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 60, seed=1))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8 if cfg.key_dtype == "e4m3" else pu.TOL_BF16)


FLAT_BF16 = CONFIGS["cfg2"].replace(name="flat_bf16", L=5000, Ksp=512, W=256, R=1, seed=14, hi_enable=False)
FLAT_FP8 = CONFIGS["cfg3"].replace(name="flat_fp8", L=6000, Ksp=512, W=384, R=1, seed=15, hi_enable=False)
FLAT_SHORT = CONFIGS["cfg1"].replace(name="flat_short", hi_enable=False)          # cache <= 4096: fused kernel
FLAT_CFG1 = CONFIGS["cfg1"].replace(name="flat_cfg1", L=4600, hi_enable=False)    # 8-head indexer, dense path


@pytest.mark.parametrize("cfg", [FLAT_BF16, FLAT_FP8, FLAT_SHORT, FLAT_CFG1], ids=lambda c: c.name)
def test_flat_indexer_without_the_hierarchy(cuda_device, cfg):
    """hi_enable = 0: Eq. 7 over the whole scoring range (dense token scores + top-K for long caches)."""
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 60, seed=4))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8 if cfg.key_dtype == "e4m3" else pu.TOL_BF16)
    # flat and hierarchical agree wherever the hierarchy keeps every eligible page
    hier = PrefillWorkload(cfg.replace(hi_enable=True), cuda_device)
    hier.prepare()
    hier.index()
    t_all = (cfg.M + cfg.S // cfg.P) * cfg.P + cfg.W          # first query with more than M eligible pages
    assert torch.equal(hier.sparse_idx[:t_all], wl.sparse_idx[:t_all])


def test_prefill_query_window_with_offset_matches_whole_run(cuda_device):
    """Queries [q_pos0, q_pos0+n) scored alone (chunked prefill) give the rows of the full run."""
    cfg = SMALL_MLA.replace(R=1)
    full = PrefillWorkload(cfg, cuda_device)
    full.prepare()
    full.step()
    part = PrefillWorkload(cfg, cuda_device, q_pos0=3000, n_query=500)
    part.prepare()
    part.step()
    assert torch.equal(part.sparse_idx, full.sparse_idx[3000:3500])
    assert torch.equal(part.out[0], full.out[0][3000:3500])
    # q_chunk splits the indexer passes without changing anything
    chunked = PrefillWorkload(cfg.replace(q_chunk=1000), cuda_device)
    chunked.prepare()
    chunked.step()
    assert torch.equal(chunked.sparse_idx, full.sparse_idx) and torch.equal(chunked.out[0], full.out[0])


def test_attention_on_cache_rows_with_padding(cuda_device):
    """The latent cache may be a view of wider rows (ld_k > d_qk): same output as on packed rows, both where key tiles
    are whole window runs and where they are gathered row by row."""
    cfg = SMALL_MLA.replace(R=1)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    packed = wl.k[0]
    wide = torch.zeros((packed.shape[0], cfg.d_qk + 64), dtype=packed.dtype, device=cuda_device)
    wide[:, :cfg.d_qk] = packed
    wide[:, cfg.d_qk:] = 7.0                                           # must never be read
    view = wide[:, :cfg.d_qk]
    assert view.stride(0) == cfg.d_qk + 64
    out = torch.empty_like(wl.out[0])
    wl.ctx.sparse_attn(wl.q[0], view, view, wl.sparse_idx, wl.n_sparse, 0, wl.n_query, wl.n_key, out)
    assert wl.ctx.status() == 0
    assert torch.equal(out, wl.out[0])


def test_attention_issue_order_and_completion_barrier_give_the_same_bits(cuda_device):
    """The tcgen05 attention kernel queues the Q K^T of a tile behind the P V that frees its accumulator (same issuing
    thread, program order); LSA_TUNE_ATTN_PV_WAIT = 1 makes it wait for that P V's completion barrier instead.  Same
    arithmetic in the same order either way, so the outputs must be equal bit for bit."""
    cfg = SMALL_MLA.replace(R=1)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    fast_out, fast_lse = wl.out[0].clone(), wl.lse[0].clone()
    wl.ctx.tune(3, 1)                 # LSA_TUNE_ATTN_PV_WAIT
    wl.step()
    assert wl.ctx.status() == 0
    assert torch.equal(wl.out[0], fast_out) and torch.equal(wl.lse[0], fast_lse)


def test_rows_gathered_by_tma_gather4_give_the_same_bits(cuda_device):
    """LSA_TUNE_ATTN_GATHER = 1 fetches the scattered cache rows with tile::gather4 TMA copies instead of 16-byte
    cp.async: the same bytes land in the same places of the key tile, so prefill and decode outputs are unchanged."""
    cfg = SMALL_MLA.replace(R=1)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    out0, lse0 = wl.out[0].clone(), wl.lse[0].clone()
    wl.ctx.tune(4, 1)                 # LSA_TUNE_ATTN_GATHER
    wl.step()
    assert wl.ctx.status() == 0
    assert torch.equal(wl.out[0], out0) and torch.equal(wl.lse[0], lse0)
    dw = DecodeWorkload(SMALL_DEC, cuda_device)
    dw.prepare()
    dw.step()
    dec0 = [o.clone() for o in dw.out]
    dw.ctx.tune(4, 1)
    dw.step()
    assert dw.ctx.status() == 0
    for a, b in zip(dw.out, dec0):
        assert torch.equal(a, b)


def test_group_of_three_layers(cuda_device):
    """R = 3, the paper's MTP-style group (Sec. 3.2): one index set, three attention layers with their own caches."""
    cfg = SMALL_MLA.replace(name="mla_r3", R=3, seed=29)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 40, seed=6))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_BF16)
    assert not torch.equal(wl.out[0], wl.out[2])
    dcfg = SMALL_DEC.replace(name="dec_r3", R=3, seed=30)
    dw = DecodeWorkload(dcfg, cuda_device)
    dw.prepare()
    dw.step()
    assert dw.ctx.status() == 0
    pu.check_decode(dw, range(dcfg.batch)).assert_ok(pu.TOL_FP8)


def test_runs_are_deterministic(cuda_device):
    wl = PrefillWorkload(SMALL_FP8, cuda_device)
    wl.prepare()
    wl.step()
    idx0, out0 = wl.sparse_idx.clone(), wl.out[1].clone()
    for _ in range(3):
        wl.step()
        assert torch.equal(idx0, wl.sparse_idx) and torch.equal(out0, wl.out[1])


@pytest.mark.parametrize("key_dtype", ["e4m3", "bf16"])
def test_small_paged_decode(cuda_device, key_dtype):
    """e4m3 caches: the fine stage feeds the codes to FP8 MMAs against the query heads split into three e5m2 planes;
    bf16 caches: bf16 MMAs.  Both against the fp64 oracle."""
    cfg = SMALL_DEC.replace(name="dec_small_" + key_dtype, key_dtype=key_dtype)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8 if key_dtype == "e4m3" else pu.TOL_BF16)


@pytest.mark.parametrize("key_dtype", ["e4m3", "bf16"])
def test_flat_indexer_on_paged_caches(cuda_device, key_dtype):
    """hi_enable = 0 in decode (what the paper itself runs there): Eq. 7 over every cached token of each sequence, scored
    page by page through the page table.  Contexts on both sides of the 4096-token limit of the fused kernel; a
    sequence whose eligible pages all fit the recall budget must get the same set from the hierarchy."""
    cfg = SMALL_DEC.replace(name="dec_flat_" + key_dtype, hi_enable=False, key_dtype=key_dtype, M=64, ctx_lo=1100, ctx_hi=9000, seed=23)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8 if key_dtype == "e4m3" else pu.TOL_BF16)
    hier = DecodeWorkload(cfg.replace(hi_enable=True), cuda_device)
    hier.prepare()
    hier.index()
    assert hier.ctx.status() == 0
    ctx = wl.ctx_len.cpu().numpy()
    short = [b for b in range(cfg.batch) if (int(ctx[b]) - 1 - cfg.W) // cfg.P - cfg.S // cfg.P + 1 <= cfg.M]
    assert short, "the test wants at least one sequence whose eligible pages fit the budget"
    for b in short:
        assert torch.equal(hier.sparse_idx[b], wl.sparse_idx[b])


@pytest.mark.parametrize("mode", [1, 2])
def test_paged_fine_stage_on_tcgen05_gives_the_same_selection(cuda_device, mode):
    """The fine stage over cache pages has three forms (LSA_TUNE_FINE_PAGED_TC): 0, the default, one kernel with a
    thread-block cluster per sequence (page top-M, token scores on tcgen05, top-K, cache rows); 1: the same steps as
    three kernels; 2: the mma.sync kernels.  Same arithmetic per token up to the summation order of the heads, so the
    sets of forms 1 and 2 are compared with the oracle, and with the default form."""
    cfg = SMALL_DEC
    ref_wl = DecodeWorkload(cfg, cuda_device)
    ref_wl.prepare()
    ref_wl.step()
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.ctx.tune(5, mode)
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8)
    same = sum(int(torch.equal(wl.sparse_idx[b], ref_wl.sparse_idx[b])) for b in range(cfg.batch))
    assert same >= cfg.batch - 1       # a near-tie may flip one token of one sequence


@pytest.mark.parametrize("n_split", [1, 2, 4, 8])
def test_paged_decode_row_splits(cuda_device, n_split):
    """Each row-split count of the decode attention (blocks of one thread-block cluster merging their parts by
    log-sum-exp) matches the oracle; the split is a launch shape, not part of the result's definition."""
    cfg = SMALL_DEC
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.ctx.tune(2, n_split)          # LSA_TUNE_ATTN_SPLIT
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, n_split, m.summary())
    m.assert_ok(pu.TOL_FP8)


def test_paged_decode_tiny_contexts(cuda_device):
    """Contexts from one token up: sequences with nothing outside sink and window (no candidate page, no tile, an empty
    selection), with a window that is not yet full, and with a handful of candidate pages."""
    cfg = SMALL_DEC.replace(name="dec_tiny", batch=24, ctx_lo=1, ctx_hi=700, M=8, Ksp=256, R=1, seed=41)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    ctx = wl.ctx_len.cpu().numpy()
    assert (ctx <= cfg.S + cfg.W).any() and (ctx > cfg.S + cfg.W + cfg.P).any()
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8)
    n_sp = wl.n_sparse.cpu().numpy()
    for b in range(cfg.batch):
        assert n_sp[b] == max(0, min(cfg.Ksp, int(ctx[b]) - cfg.S - cfg.W))


def test_paged_decode_large_batch(cuda_device):
    """More sequences than half the SM count: the fine stage gives each sequence one block instead of a cluster of two
    (the block scores every kept page itself).  Short contexts: some sequences have fewer eligible pages than the
    budget, and an odd number of them (a tile with one page)."""
    cfg = SMALL_DEC.replace(name="dec_wide", batch=320, ctx_lo=700, ctx_hi=1600, M=8, Ksp=256, R=1, seed=19)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, [0, 1, 17, 150, 318, 319])
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8)


def test_decode_step_replays_from_a_cuda_graph(cuda_device):
    """lsa_layer_group on a side stream makes no synchronising call: a decode step captures into a CUDA graph, and
    the replay writes the bytes of the eager step."""
    side = torch.cuda.Stream(device=cuda_device)
    with torch.cuda.stream(side):
        wl = DecodeWorkload(SMALL_DEC, cuda_device)
        wl.prepare()
        wl.step()
        wl.step()
        side.synchronize()
        want = [o.clone() for o in wl.out] + [wl.sparse_idx.clone()]
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            wl.step()
        for o in wl.out:
            o.zero_()
        wl.sparse_idx.zero_()
        graph.replay()
        side.synchronize()
        assert wl.ctx.status() == 0
        for a, b in zip(want, wl.out + [wl.sparse_idx]):
            assert torch.equal(a, b)


def test_decode_split_count_is_checked(cuda_device):
    cfg = SMALL_DEC
    if cfg.H != 64:
        pytest.skip("cluster splits belong to the 64-head kernel")
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.ctx.tune(2, 3)                # three blocks do not divide the 64 heads evenly
    with pytest.raises(binding.LsaError):
        wl.step()


def test_convert_lists_physical_rows(cuda_device):
    cfg = SMALL_DEC
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.index()
    ld = cfg.S + cfg.Ksp + cfg.W
    rows = torch.empty((cfg.batch, ld), dtype=torch.int32, device=cuda_device)
    n_rows = torch.empty((cfg.batch,), dtype=torch.int32, device=cuda_device)
    runs = torch.empty((cfg.batch, 4), dtype=torch.int32, device=cuda_device)
    wl.ctx.convert(wl.sparse_idx, wl.n_sparse, 0, cfg.batch, rows, n_rows, runs, wl.page_table, wl.ctx_len)
    table, ctx = pu.to_np(wl.page_table), pu.to_np(wl.ctx_len)
    for b in range(cfg.batch):
        t = int(ctx[b]) - 1
        n_sp = int(wl.n_sparse[b])
        S_t = orc.index_set(t, cfg.S, cfg.W, pu.to_np(wl.sparse_idx[b])[:n_sp])
        want = orc.paged_rows(S_t, table[b], cfg.kv_page)
        got = pu.to_np(rows[b])
        assert int(n_rows[b]) == len(want) and np.array_equal(got[:len(want)], want) and (got[len(want):] == -1).all()
        r = pu.to_np(runs[b])
        assert list(r[:3]) == [cfg.S, n_sp, cfg.W]
        assert r[3] == 1 + int((np.diff(want) != 1).sum())
        # the window is whole-page runs: far fewer breaks than rows
        assert r[3] <= n_sp + cfg.W // cfg.kv_page + 3


# ---------------------------------------------------------------- recall budgets beyond 4096 tokens
@pytest.mark.parametrize("base", ["fp8", "bf16"])
def test_large_recall_budget(cuda_device, base):
    """M * P = 8192 candidate tokens per query (twice what the fused fine kernel holds): page list, fine scores through
    the workspace and the standalone top-K give the oracle's pages and tokens, in one pass and in query chunks."""
    src = CONFIGS["cfg3"] if base == "fp8" else CONFIGS["cfg2"]
    cfg = src.replace(name=f"big_{base}", L=20000, P=64, M=128, Ksp=1024, W=384, R=1, seed=27, q_chunk=0)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    pages = torch.full((wl.n_query, cfg.M), -7, dtype=torch.int32, device=cuda_device)
    wl.index(pages)
    assert wl.ctx.status() == 0
    qs = pu.boundary_queries(cfg, 0, cfg.L, 40, seed=3)
    m = pu.check_prefill(wl, qs, check_attention=False, pages=pages)
    print(cfg.name, m.summary())
    assert m.summary()["mean_overlap"] >= pu.MIN_OVERLAP and m.summary()["page_sets_differ"] == 0
    whole = wl.sparse_idx.clone()
    del wl
    wl2 = PrefillWorkload(cfg.replace(q_chunk=3000), cuda_device)
    wl2.prepare()
    wl2.step()
    assert torch.equal(wl2.sparse_idx, whole)
    m2 = pu.check_prefill(wl2, qs[-6:], check_attention=True)
    m2.assert_ok(pu.TOL_FP8 if base == "fp8" else pu.TOL_BF16)


# ---------------------------------------------------------------- host-buffer entry point
@pytest.mark.parametrize("q_pos0", [0, 2100])
def test_layer_group_from_host_buffers_equals_device_run(cuda_device, q_pos0):
    """lsa_layer_group_host (queries in pinned host memory, staged through the device in passes, copies overlapping
    kernels) returns the bytes of the device-resident run, for a pass size that leaves a ragged last pass and needs
    every staging buffer several times; also for a chunk of queries that starts inside the sequence."""
    cfg = SMALL_FP8.replace(name="host_small", L=5000, R=2, seed=23)
    wl = PrefillWorkload(cfg, cuda_device, with_lse=False, q_pos0=q_pos0, n_query=cfg.L - q_pos0)
    wl.prepare()
    wl.step()
    torch.cuda.synchronize()
    sq = 768
    stage = [torch.empty(binding.host_stage_bytes(wl.params, sq), dtype=torch.uint8, device=cuda_device) for _ in range(2)]
    q_idx_h, w_h = wl.q_idx.cpu().pin_memory(), wl.w.cpu().pin_memory()
    q_h = [q.cpu().pin_memory() for q in wl.q]
    out_h = [torch.zeros(o.shape, dtype=o.dtype).pin_memory() for o in wl.out]
    for _ in range(2):   # twice: the second call reuses events and staging areas left by the first
        wl.ctx.layer_group_host(q_idx_h, w_h, wl.keys["k"], wl.keys.get("scale"), wl.kmean, wl.q_pos0, wl.n_query, wl.n_key, q_h,
                                wl.k, wl.v, out_h, sq, stage)
        torch.cuda.synchronize()
        assert wl.ctx.status() == 0
        for oh, o in zip(out_h, wl.out):
            assert torch.equal(oh, o.cpu())


# ---------------------------------------------------------------- decode-step cache maintenance
def test_append_tokens_then_decode(cuda_device):
    """37 decode steps of cache maintenance (crossing sub-block and page boundaries): the stored codes and scales are
    the oracle's, the means equal both the oracle's and a rebuild by lsa_block_means, the attention rows land where
    the page table says, and a decode step on the grown caches matches the oracle."""
    n_add = 37
    cfg = SMALL_DEC.replace(name="dec_append", ctx_grow=n_add + 3, R=2, seed=17)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    ctx0 = pu.to_np(wl.ctx_len).astype(np.int64)
    table = pu.to_np(wl.page_table)
    # oracle-side logical caches of every sequence, with room to grow
    host = []
    k_pool0, s_pool0 = pu.to_np(wl.keys["k"]), pu.to_np(wl.keys["scale"])
    for b in range(cfg.batch):
        n0 = int(ctx0[b])
        rows = orc.paged_rows(np.arange(n0), table[b], cfg.kv_page)
        codes = np.zeros((n0 + n_add, cfg.d_I), np.uint8)
        scales = np.ones(n0 + n_add, np.float32)
        codes[:n0], scales[:n0] = k_pool0[rows], s_pool0[rows]
        km = np.zeros((-(-(n0 + n_add) // cfg.B), cfg.d_I))
        km[:-(-n0 // cfg.B)] = orc.block_means(orc.dequant_keys(codes[:n0], scales[:n0]), cfg.B)
        host.append([codes, scales, km, n0])
    g = torch.Generator(device=cuda_device)
    g.manual_seed(1234)
    kv_rows = {}
    for step in range(n_add):
        k_new = (torch.randn((cfg.batch, cfg.d_I), generator=g, device=cuda_device) / math.sqrt(cfg.d_I)).to(torch.bfloat16)
        if step == 5:
            k_new[1] = 0                                   # a zero key: scale 1, codes 0
        kv_new = [torch.randn((cfg.batch, cfg.d_qk), generator=g, device=cuda_device).to(torch.bfloat16) for _ in range(cfg.R)]
        wl.ctx.append(k_new, wl.keys["k"], wl.keys["scale"], wl.kmean, wl.page_table, wl.ctx_len, wl.ctx_len, kv_new, wl.k)
        kn = pu.to_np(k_new)
        for b in range(cfg.batch):
            h = host[b]
            kv_rows[(b, h[3])] = [pu.to_np(x[b]) for x in kv_new]
            h[3] = orc.append_token(h[0], h[1], h[2], h[3], kn[b], cfg.B)
    assert wl.ctx.status() == 0
    assert np.array_equal(pu.to_np(wl.ctx_len), ctx0 + n_add)
    k_pool, s_pool, km_pool = pu.to_np(wl.keys["k"]), pu.to_np(wl.keys["scale"]), pu.to_np(wl.kmean).astype(np.float64)
    # a rebuild of the mean cache from the grown pools
    km2 = torch.zeros_like(wl.kmean)
    wl.ctx.block_means(wl.keys["k"], wl.keys.get("scale"), 0, km2, wl.page_table, wl.ctx_len)
    km2 = pu.to_np(km2).astype(np.float64)
    spp_kv = cfg.kv_page // cfg.B
    n_diff = n_tot = 0
    for b in range(cfg.batch):
        codes, scales, km, n = host[b]
        rows = orc.paged_rows(np.arange(n), table[b], cfg.kv_page)
        assert np.array_equal(k_pool[rows], codes[:n]) and np.array_equal(s_pool[rows], scales[:n])
        subs = np.arange(-(-n // cfg.B))
        mrows = table[b][subs * cfg.B // cfg.kv_page].astype(np.int64) * spp_kv + (subs * cfg.B % cfg.kv_page) // cfg.B
        assert np.array_equal(km_pool[mrows], km2[mrows])                    # appended == rebuilt, bit for bit
        d = np.abs(km_pool[mrows] - km[:len(subs)])
        # fp32 against fp64 accumulation: at most one bf16 ulp of the mean, or the fp32 error of the sum when it cancels
        assert (d <= np.abs(km[:len(subs)]) * 2.0 ** -7 + 1e-6).all()
        n_diff += int((d > 0).sum())
        n_tot += d.size
        for pos in range(int(ctx0[b]), n):
            r = int(orc.paged_rows(np.array([pos]), table[b], cfg.kv_page)[0])
            for layer in range(cfg.R):
                assert np.array_equal(pu.to_np(wl.k[layer][r]), kv_rows[(b, pos)][layer])
    assert n_diff < 0.005 * n_tot
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    print(cfg.name, m.summary())
    m.assert_ok(pu.TOL_FP8)


# ---------------------------------------------------------------- MinMax pooling (Eq. 13)
@pytest.mark.parametrize("base", ["fp8", "bf16"])
def test_minmax_cache_and_selection(cuda_device, base):
    """The extrema cache equals the oracle's (an extremum is a key value: one rounding), and the two-stage selection
    with Eq. 13 page scores picks the oracle's pages and tokens."""
    if base == "fp8":
        cfg = SMALL_FP8.replace(name="mm_fp8", pooling="minmax", R=1)
    else:
        cfg = CONFIGS["cfg1"].replace(name="mm_bf16", pooling="minmax", L=1500, seed=41)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    k_hat = (orc.dequant_keys(pu.to_np(wl.keys["k"]), pu.to_np(wl.keys["scale"])) if "scale" in wl.keys
             else pu.to_np(wl.keys["k"]).astype(np.float64))
    kmax, kmin = orc.block_minmax(k_hat, cfg.B)
    got = pu.to_np(wl.kmean).astype(np.float64)
    want = np.concatenate([kmax, kmin], axis=1)
    # e4m3: the kernel rounds code x scale to fp32 before bf16, the oracle rounds the exact product once
    diff = np.abs(got - want)
    assert (diff <= np.abs(want) * 2.0 ** -7).all() and (diff > 0).mean() < 2e-3
    pages = torch.full((wl.n_query, cfg.M), -7, dtype=torch.int32, device=cuda_device)
    wl.index(pages)
    assert wl.ctx.status() == 0
    m = pu.check_prefill(wl, pu.boundary_queries(cfg, 0, cfg.L, 60, seed=5), check_attention=False, pages=pages)
    print(cfg.name, m.summary())
    assert m.summary()["mean_overlap"] >= pu.MIN_OVERLAP


def test_minmax_rejects_paged_caches(cuda_device):
    p = binding.make_params(SMALL_DEC.replace(pooling="minmax"))
    with pytest.raises(binding.LsaError):
        binding.workspace_bytes(p, 8, 4096, 8)


# ---------------------------------------------------------------- edge cases and errors
def test_short_sequences_and_empty_calls(cuda_device):
    cfg = CONFIGS["cfg1"].replace(L=100, name="short")            # L < S + W: every query sees [0, t]
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert int(wl.n_sparse.max()) == 0 and (wl.sparse_idx == -1).all()
    m = pu.check_prefill(wl, range(cfg.L))
    m.assert_ok(pu.TOL_BF16)
    # zero queries: nothing is launched, nothing fails
    n0 = wl.ctx.launch_count()
    wl.ctx.index(wl.q_idx, wl.w, wl.keys["k"], None, wl.kmean, 0, 0, cfg.L, wl.sparse_idx, wl.n_sparse)
    assert wl.ctx.launch_count() == n0 and wl.ctx.status() == 0


def test_full_candidate_budget_selects_every_candidate(cuda_device):
    """Ksp >= number of candidates: S_t = [0, t] and the result is dense causal attention."""
    cfg = CONFIGS["cfg1"].replace(L=600, Ksp=512, M=8, name="dense")
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    n_sp = pu.to_np(wl.n_sparse)
    for t in range(cfg.L):
        assert n_sp[t] == max(0, t - cfg.W - cfg.S + 1)
    q, k, v = pu.to_np(wl.q[0]).astype(np.float64), pu.to_np(wl.k[0]).astype(np.float64), pu.to_np(wl.v[0]).astype(np.float64)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k)[None, None].expand(1, cfg.H, cfg.L, cfg.d_qk)
    tv = torch.from_numpy(v)[None, None].expand(1, cfg.H, cfg.L, cfg.d_v)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=cfg.sm_scale)[0]
    got = torch.from_numpy(pu.to_np(wl.out[0])).permute(1, 0, 2).to(torch.float64)
    assert (got - ref).abs().max() <= 2e-2
    assert ((got - ref).norm() / ref.norm()) <= 5e-3


def test_errors_are_codes_not_crashes(cuda_device):
    cfg = CONFIGS["cfg1"]
    bad = binding.make_params(cfg.replace(H_I=12))
    with pytest.raises(binding.LsaError) as e:
        binding.workspace_bytes(bad, 10, 100)
    assert e.value.code == -2
    wl = PrefillWorkload(cfg.replace(L=256, name="err"), cuda_device)
    with pytest.raises(binding.LsaError) as e:                     # queries beyond the cache
        wl.ctx.index(wl.q_idx, wl.w, wl.keys["k"], None, wl.kmean, 200, 100, 256, wl.sparse_idx, wl.n_sparse)
    assert e.value.code == -1
    small_ws = binding.Context(wl.params, 1, 64, device=cuda_device)
    with pytest.raises(binding.LsaError) as e:                     # workspace sized for a smaller problem
        small_ws.index(wl.q_idx, wl.w, wl.keys["k"], None, wl.kmean, 0, 256, 256, wl.sparse_idx, wl.n_sparse)
    assert e.value.code == -3
    assert wl.ctx.status() == 0
