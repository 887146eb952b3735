"""Pins for the oracle's number formats and cache arithmetic (CPU only)."""
import numpy as np
import torch

from oracle import lsa_oracle as orc
from paper_2608_01662_b200 import inputs
from paper_2608_01662_b200.configs import CONFIGS


def test_e4m3_decode_matches_library_for_all_256_codes():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = orc.e4m3_decode(codes)
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert np.signbit(got[0x80]) and got[0x80] == 0.0
    assert got[0x7e] == 448.0 and got[0x01] == 2.0 ** -9


def test_e4m3_values_are_exact_in_bf16():
    # every finite e4m3 value has 4 significant bits: widening to bf16 loses nothing
    v = orc.e4m3_decode(np.arange(256, dtype=np.uint8))
    v = v[~np.isnan(v)]
    assert np.array_equal(orc.bf16_round(v), v)


def test_bf16_round_matches_library_rounding():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000), rng.standard_normal(2000) * 1e-3,
                        rng.standard_normal(2000) * 1e3, [0.0, 1.0, -1.0, 1.00390625, 1.01171875]])
    x32 = x.astype(np.float32).astype(np.float64)       # fp32-exact inputs: torch rounds fp32 -> bf16 RNE
    ref = torch.from_numpy(x32).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.bf16_round(x32), ref)
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert orc.bf16_round(np.array([1.00390625]))[0] == 1.0
    assert orc.bf16_round(np.array([1.01171875]))[0] == 1.015625


def test_quantizer_roundtrip_error_and_saturation():
    g = torch.Generator().manual_seed(1)
    k = torch.randn(512, 128, generator=g) * 0.1
    k[7] = 0
    codes, scale = inputs.quantize_e4m3(k)
    assert scale[7] == 1.0
    deq = orc.dequant_keys(codes.numpy(), scale.numpy())
    assert not np.isnan(deq).any()
    amax = k.abs().amax(dim=1).numpy().astype(np.float64)
    # e4m3 has 3 mantissa bits: relative step 2^-3, so |err| <= amax * 2^-4 (plus subnormal floor)
    assert (np.abs(deq - k.numpy().astype(np.float64)).max(axis=1) <= amax * 2.0 ** -4 + 1e-12).all()
    # the largest element of each row maps onto +-448 exactly
    assert (np.abs(orc.e4m3_decode(codes.numpy())).max(axis=1)[amax > 0] == 448.0).all()


def test_block_means_against_plain_loops_and_partial_tail():
    rng = np.random.default_rng(3)
    k = rng.standard_normal((37, 5))
    km = orc.block_means(k, 8, round_bf16=False)
    assert km.shape == (5, 5)
    for n in range(5):
        rows = [k[s] for s in range(n * 8, min(n * 8 + 8, 37))]
        for d in range(5):
            assert abs(km[n, d] - sum(r[d] for r in rows) / len(rows)) < 1e-15
    # B = 1: the mean cache is the key cache (the "size 1" column of the pooling ablation)
    assert np.array_equal(orc.block_means(k, 1, round_bf16=False), k)
    # rounded variant lands on the bf16 grid
    kr = orc.block_means(k, 8)
    assert np.array_equal(kr, torch.from_numpy(kr).to(torch.bfloat16).to(torch.float64).numpy())


def test_paper_closed_forms():
    """Arithmetic facts the paper states (see tests/golden/paper_facts.txt)."""
    facts = {}
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                key, val = line.split("=")[0].strip(), line.split("=")[1].split("#")[0].strip()
                facts[key] = float(val)
    c = CONFIGS["cfg2"]
    assert c.d_qk * 2 == facts["latent_bytes_bf16"]                    # one latent KV entry
    assert abs((1 - 2048 / 131072) * 100 - facts["sparsity_pct_K2048_128K"]) < 0.05
    assert 1024 * 128 == facts["recall_tokens_M1024_P128"]
    assert 16 + 1024 + 1024 <= facts["K_total"] + 16                  # K = K_sink + K_swa + K_sparse
    # gather efficiency estimate of Sec. 2.3: 3 of ~50 cachelines in flight, 75 % packed
    assert abs(3 / 50 * (1152 / (3 * 512)) * 100 - facts["sfa_hbm_pct"]) < 0.05


def test_generators_are_deterministic_and_chunk_consistent():
    cfg = CONFIGS["cfg1"]
    q1, w1 = inputs.indexer_queries(cfg, 0, 64, "cpu")
    q2, w2 = inputs.indexer_queries(cfg, 32, 16, "cpu")
    assert torch.equal(q1[32:48], q2) and torch.equal(w1[32:48], w2)
    k = inputs.indexer_keys(CONFIGS["cfg3"].replace(L=256), 256, "cpu")
    assert k["k"].dtype == torch.uint8 and k["scale"].shape == (256,)
    ctx, table, n_pg = inputs.decode_layout(CONFIGS["cfg4"].replace(batch=4, ctx_lo=100, ctx_hi=300), "cpu")
    used = table[table >= 0]
    assert used.numel() == n_pg and torch.equal(torch.sort(used).values, torch.arange(n_pg, dtype=torch.int32))
    assert ((ctx >= 100) & (ctx <= 300)).all()


# ---------------------------------------------------------------- e4m3 encoding and the append-token maintenance
def test_e4m3_encode_round_trips_every_code_and_matches_a_library_cast():
    import torch
    codes = np.arange(256, dtype=np.uint8)
    finite = codes[(codes & 0x7f) != 0x7f]
    vals = orc.e4m3_decode(finite)
    back = orc.e4m3_encode(vals)
    keep = finite != 0x80                                   # -0 encodes as 0x80 as well: compare values there
    assert np.array_equal(back[keep], finite[keep]) and orc.e4m3_decode(back[~keep])[0] == 0.0
    # an independent implementation of the same rounding: torch's float8_e4m3fn cast (saturation applied by hand)
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(20000) * 100.0, rng.standard_normal(20000) * 0.01,
                        np.array([0.0, 448.0, 460.0, -1000.0, 2.0 ** -9, 2.0 ** -10, 1.5 * 2.0 ** -9, 17.0, 19.0, 0.0625 * 1.0625])])
    x32 = x.astype(np.float32)
    want = torch.from_numpy(x32).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = orc.e4m3_encode(x32)
    same_value = orc.e4m3_decode(got) == orc.e4m3_decode(want)      # +0 / -0 may differ in sign bit only
    assert same_value.all()
    # ties go to the even mantissa: 17 lies between 16 (m=0) and 18 (m=1); 19 between 18 (m=1) and 20 (m=2)
    assert orc.e4m3_decode(orc.e4m3_encode(np.array([17.0, 19.0]))).tolist() == [16.0, 20.0]


def test_quantize_token_scale_and_error_bound():
    rng = np.random.default_rng(6)
    k = (rng.standard_normal(128) * 0.3).astype(np.float32)
    codes, scale = orc.quantize_token(k)
    assert scale == np.float32(np.abs(k).max() / np.float32(448.0))
    err = np.abs(orc.e4m3_decode(codes) * float(scale) - k)
    # relative step of e4m3 is 2^-3 for normal values: half a step, plus the subnormal floor 2^-10 * scale
    assert (err <= np.maximum(np.abs(k) * 2.0 ** -4, 2.0 ** -10 * float(scale)) * 1.0001).all()
    assert np.abs(orc.e4m3_decode(codes)).max() == 448.0
    z, s1 = orc.quantize_token(np.zeros(16, np.float32))
    assert s1 == 1.0 and (z == 0).all()


def test_append_token_equals_rebuilding_the_caches():
    """Appending tokens one at a time leaves the caches exactly as quantising all keys and calling block_means on
    the whole sequence would (the scale is per token, a mean is a function of its sub-block alone)."""
    rng = np.random.default_rng(7)
    d, B, n0, n_add = 16, 8, 21, 30
    keys = (rng.standard_normal((n0 + n_add, d)) * 0.2).astype(np.float32)
    codes = np.zeros((n0 + n_add, d), np.uint8)
    scales = np.ones(n0 + n_add, np.float32)
    for i in range(n0):
        codes[i], scales[i] = orc.quantize_token(keys[i])
    km = np.zeros((-(-(n0 + n_add) // B), d))
    km[:-(-n0 // B)] = orc.block_means(orc.dequant_keys(codes[:n0], scales[:n0]), B)
    n = n0
    for i in range(n_add):
        n = orc.append_token(codes, scales, km, n, keys[n], B)
        want = orc.block_means(orc.dequant_keys(codes[:n], scales[:n]), B)
        assert np.array_equal(km[:want.shape[0]], want)
    full_codes = np.stack([orc.quantize_token(k)[0] for k in keys])
    assert n == n0 + n_add and np.array_equal(codes, full_codes)
    # bf16 cache form
    kb = orc.bf16_round(keys.astype(np.float64))
    cache = np.zeros_like(kb)
    cache[:n0] = kb[:n0]
    km2 = np.zeros_like(km)
    km2[:-(-n0 // B)] = orc.block_means(kb[:n0], B)
    n = n0
    for i in range(n_add):
        n = orc.append_token(cache, None, km2, n, kb[n], B)
    assert np.array_equal(km2, orc.block_means(kb, B))
