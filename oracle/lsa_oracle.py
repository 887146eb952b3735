"""CPU oracle for the LongCat-Sparse-Attention indexer + sparse-attention forward.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition the CUDA
library is checked against.  It may be imported by the test-suite, by the smoke
check and by the benchmark's CPU-baseline leg, never by the product path, and it
shares no code, table or constant with the CUDA sources.

All arithmetic is float64 on the *stored* input values (bf16 / e4m3 values are
first widened exactly to float64).  Positions are 0-indexed; the paper writes
them 1-indexed.  One function per step, in the paper's order:

  e4m3_decode, dequant_keys      stored fp8 keys -> real values (FP8 indexer, Sec. 2.2)
  e4m3_encode, quantize_token    real key -> stored fp8 code and per-token scale (fp32 decision)
  block_means                    per-dimension sub-block mean keys (Sec. 3.3, stage 1)
  block_minmax, page_scores_minmax   the MinMax pooling variant (Eq. 13)
  append_token                   cache maintenance of one decode step (new key, its sub-block mean)
  indexer_scores                 Eq. 1 / Eq. 11
  page_scores                    Eq. 9
  top_k                          arg-topK with the total order (score desc, id asc)
  candidate_range, eligible_pages  Eq. 6-7 scoring range, Eq. 10 page range
  select_sparse                  Eq. 9-12 (hierarchical) or Eq. 7 (flat)
  index_set                      Eq. 6:  sink U window U sparse
  attend                         Eq. 3 on an explicit index set (absorbed-MQA: one K/V row
                                 shared by every head)
  select_fp32                    the selection step alone on given float32 scores
  paged_rows / gather_paged      logical position -> physical cache row (paged caches, App. B)

Pins (tests/test_oracle_*.py) check every function against something outside
this file: brute-force loops, full sorts, torch/scipy library routines, closed
forms and the equivalences the paper states.  No function here is unpinned.

Readings taken where the paper is silent, and that matter for the arithmetic, are
stated in the docstrings below.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# number formats
# ----------------------------------------------------------------------------


def e4m3_decode(codes):
    """OCP FP8 E4M3 ("fn": no infinities, 0x7f/0xff are NaN) code -> float64.

    sign(1) exponent(4, bias 7) mantissa(3); exponent 0 is subnormal
    (m/8 * 2^-6); largest finite value 448.
    """
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    sub = (m / 8.0) * 2.0 ** -6
    val = np.where(e == 0, sub, normal)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def e4m3_encode(x):
    """Real value -> OCP FP8 E4M3 code, round to nearest (ties to the even mantissa), saturating at +-448.

    Written as a search over the 127 non-negative finite code values, so that it shares nothing with e4m3_decode's
    closed form except the table that function produces; NaN is not expected.
    """
    x = np.asarray(x, dtype=np.float64)
    mags = e4m3_decode(np.arange(0, 127, dtype=np.uint8))          # codes 0x00..0x7e, ascending values 0..448
    a = np.minimum(np.abs(x), 448.0)
    hi = np.searchsorted(mags, a, side="left").clip(0, 126)        # first code value >= a
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = mags[hi] - a, a - mags[lo]
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))     # tie: the code with the even mantissa bit
    code = np.where(pick_lo, lo, hi).astype(np.uint8)
    return np.where(np.signbit(x), code | 0x80, code).astype(np.uint8)


def quantize_token(k_row):
    """One indexer key (any real dtype) -> (e4m3 codes uint8 [d], fp32 scale): scale = amax / 448 (1 for a zero row),
    code = RNE(k / scale).  The scale and the quotient are fp32 values, as on the device: a quantised code is an
    integer decision and both sides take it in the same precision."""
    k = np.asarray(k_row, dtype=np.float32)
    amax = np.float32(np.abs(k).max()) if k.size else np.float32(0)
    scale = np.float32(amax / np.float32(448.0)) if amax > 0 else np.float32(1.0)
    return e4m3_encode((k / scale).astype(np.float32)), scale


def append_token(k_codes, k_scale, km, n_key, k_new, B):
    """Cache maintenance of one decode step for one sequence (Sec. 3.3: the mean keys are maintained with the cache):
    the new token's indexer key is quantised and stored at position n_key, and the mean of the sub-block that holds
    it is recomputed over the tokens now present.  Arrays are logical (unpaged) and large enough; returns n_key + 1.
    With k_scale None the cache holds real (bf16) keys and k_new is stored as is."""
    if k_scale is not None:
        codes, scale = quantize_token(k_new)
        k_codes[n_key] = codes
        k_scale[n_key] = scale
    else:
        k_codes[n_key] = k_new
    n = n_key // B
    lo, hi = n * B, n_key + 1
    blk = dequant_keys(k_codes[lo:hi], k_scale[lo:hi]) if k_scale is not None else np.asarray(k_codes[lo:hi], np.float64)
    km[n] = bf16_round(blk.sum(axis=0) / (hi - lo))
    return n_key + 1


def dequant_keys(k_codes, k_scale):
    """Stored fp8 indexer keys -> real keys: decode(code) * per-token scale."""
    return e4m3_decode(k_codes) * np.asarray(k_scale, dtype=np.float64)[:, None]


def bf16_round(x):
    """Round float64 values to the nearest bfloat16 value (ties to even), as float64.

    Done on the float64 value directly (one rounding), by scaling the value so
    that the bf16 grid (8 significant bits) becomes the integers.  Finite,
    normal-range inputs only, which is all the path produces.
    """
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = x != 0
    _, ex = np.frexp(x[nz])  # x = mant * 2^ex, 0.5 <= |mant| < 1
    # 8 significant bits -> quantum 2^(ex-8)
    q = np.exp2((ex - 8).astype(np.float64))
    out[nz] = np.rint(x[nz] / q) * q  # np.rint rounds half to even
    return out


# ----------------------------------------------------------------------------
# stage 0: sub-block mean keys (Sec. 3.3 "Stage 1", first paragraph)
# ----------------------------------------------------------------------------


def block_means(k_hat, B, round_bf16=True):
    """k_mean[n] = per-dimension mean of the keys of sub-block n (B tokens).

    A trailing partial sub-block averages the tokens present.  The cache stores
    bf16, so the mean is rounded to bf16 (round_bf16=False keeps the exact mean,
    for the linearity pins).
    """
    k_hat = np.asarray(k_hat, dtype=np.float64)
    n_key, d = k_hat.shape
    n_sub = -(-n_key // B)
    km = np.zeros((n_sub, d), dtype=np.float64)
    for n in range(n_sub):
        blk = k_hat[n * B:min((n + 1) * B, n_key)]
        km[n] = blk.sum(axis=0) / blk.shape[0]
    return bf16_round(km) if round_bf16 else km


def block_minmax(k_hat, B, round_bf16=True):
    """Per-dimension extrema of the keys of each sub-block (pooling variant of Sec. 5 "Pooling method", Eq. 13):
    k_max[n, d] = max_{s in sub-block n} k[s, d],  k_min[n, d] = min likewise.

    A trailing partial sub-block takes the extrema of the tokens present.  Returns (k_max, k_min), each
    [ceil(n_key/B), d]; the cache stores bf16 (an extremum is one of the key values, rounded once).
    """
    k_hat = np.asarray(k_hat, dtype=np.float64)
    n_key, d = k_hat.shape
    n_sub = -(-n_key // B)
    kmax = np.zeros((n_sub, d), dtype=np.float64)
    kmin = np.zeros((n_sub, d), dtype=np.float64)
    for n in range(n_sub):
        blk = k_hat[n * B:min((n + 1) * B, n_key)]
        kmax[n] = blk.max(axis=0)
        kmin[n] = blk.min(axis=0)
    if round_bf16:
        return bf16_round(kmax), bf16_round(kmin)
    return kmax, kmin


# ----------------------------------------------------------------------------
# scores
# ----------------------------------------------------------------------------


def indexer_scores(q_I, w, keys):
    """Eq. 1:  I[s] = sum_j w[j] * ReLU(q_I[j] . keys[s])   for every row s of `keys`.

    q_I [H_I, d_I], w [H_I], keys [n, d_I]  ->  [n]
    """
    q_I = np.asarray(q_I, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    keys = np.asarray(keys, dtype=np.float64)
    dots = keys @ q_I.T                      # [n, H_I]
    return np.maximum(dots, 0.0) @ w         # [n]


def page_scores(q_I, w, km, P, B, pages):
    """Eq. 9:  I_page[p] = sum_j w[j] * sum_{n in page p} ReLU(q_I[j] . k_mean[n]).

    Every existing sub-block of the page takes part (a trailing page may hold
    fewer than P/B).  Returns one score per entry of `pages`.
    """
    km = np.asarray(km, dtype=np.float64)
    spp = P // B
    out = np.zeros(len(pages), dtype=np.float64)
    for i, p in enumerate(pages):
        blk = km[p * spp:min((p + 1) * spp, km.shape[0])]
        # sum over sub-blocks of the per-sub-block Eq.-1-style score
        out[i] = indexer_scores(q_I, w, blk).sum()
    return out


def page_scores_minmax(q_I, w, kmax, kmin, P, B, pages):
    """Eq. 13 in place of the mean-pooled dot product of Eq. 9: for sub-block n and head j

        s~[n, j] = sum_d max(q_I[j, d] * k_max[n, d], q_I[j, d] * k_min[n, d]),

    an upper bound of every token score q_I[j] . k[s] inside the sub-block, and
    I_page[p] = sum_j w[j] * sum_{n in page p} ReLU(s~[n, j]).  (The paper's inner sum runs to "N"; it is the
    sum over the sub-blocks of the page, as in Eq. 9.)  Returns one score per entry of `pages`.
    """
    q_I = np.asarray(q_I, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    kmax = np.asarray(kmax, dtype=np.float64)
    kmin = np.asarray(kmin, dtype=np.float64)
    spp = P // B
    out = np.zeros(len(pages), dtype=np.float64)
    for i, p in enumerate(pages):
        lo, hi = p * spp, min((p + 1) * spp, kmax.shape[0])
        total = 0.0
        for n in range(lo, hi):
            # [H_I, d]: the larger of the two products, dimension by dimension
            s_tilde = np.maximum(q_I * kmax[n][None, :], q_I * kmin[n][None, :]).sum(axis=1)
            total += float((w * np.maximum(s_tilde, 0.0)).sum())
        out[i] = total
    return out


# ----------------------------------------------------------------------------
# selection
# ----------------------------------------------------------------------------


def top_k(scores, ids, k):
    """The k entries largest under the total order (score descending, id ascending).

    +0.0 and -0.0 compare equal (IEEE).  Returns the chosen ids in ascending
    order.  If k >= len(ids) everything is chosen.
    """
    scores = np.asarray(scores)
    ids = np.asarray(ids, dtype=np.int64)
    if k <= 0 or ids.size == 0:
        return np.zeros(0, dtype=np.int64)
    # full sort: primary key -score (ascending), secondary key id (ascending)
    order = np.lexsort((ids, -scores))
    return np.sort(ids[order[:k]])


def candidate_range(t, S, W):
    """Scoring range of query t under Eq. 7: positions outside sink and window.

    sink = [0, S), window = [t-W+1, t]  ->  candidates = [S, t-W]; (lo, hi)
    with hi < lo meaning empty.
    """
    return S, t - W


def eligible_pages(t, S, W, P):
    """Pages that hold at least one candidate position of query t."""
    lo, hi = candidate_range(t, S, W)
    if hi < lo:
        return np.zeros(0, dtype=np.int64)
    return np.arange(lo // P, hi // P + 1, dtype=np.int64)


def select_sparse(t, q_I, w, k_hat, km, *, P, B, M, Ksp, S, W, hi_enable=True, minmax=None):
    """S_sparse of query t (absolute position) and the recalled pages.

    Stage 1 (Eq. 9-10): if more than M pages are eligible, keep the M with the
    largest page score.  Stage 2 (Eq. 11-12): score the candidate tokens of the
    kept pages with Eq. 1 and keep the Ksp largest.  With hi_enable False, or
    when at most M pages are eligible, every eligible page is kept, which is
    the flat selection of Eq. 7.

    k_hat [n_key, d_I] real key values, km [ceil(n_key/B), d_I] mean cache.  minmax = (k_max, k_min) switches
    stage 1 to the MinMax pooling of Eq. 13 (km is then unused).
    Returns (sparse positions ascending, kept pages ascending).
    """
    lo, hi = candidate_range(t, S, W)
    E = eligible_pages(t, S, W, P)
    if E.size == 0:
        return np.zeros(0, dtype=np.int64), E
    if hi_enable and E.size > M:
        if minmax is not None:
            pages = top_k(page_scores_minmax(q_I, w, minmax[0], minmax[1], P, B, E), E, M)
        else:
            pages = top_k(page_scores(q_I, w, km, P, B, E), E, M)
    else:
        pages = E
    cand = np.concatenate([np.arange(max(lo, p * P), min(hi, p * P + P - 1) + 1, dtype=np.int64)
                           for p in pages])
    I = indexer_scores(q_I, w, np.asarray(k_hat)[cand])
    return top_k(I, cand, Ksp), pages


def index_set(t, S, W, sparse):
    """Eq. 6: sink U window U sparse for query t, as one ascending position list.

    Early queries: sink = [0, min(S, t+1)), window = [max(S, t-W+1), t].
    """
    sink = np.arange(0, min(S, t + 1), dtype=np.int64)
    win = np.arange(max(S, t - W + 1), t + 1, dtype=np.int64)
    return np.concatenate([sink, np.asarray(sparse, dtype=np.int64), win])


def select_fp32(scores, cand_pos, t, k, *, apply_range, S=0, W=0):
    """The selection step alone, on float32 scores compared as float32.

    scores [n_cand] float32; column c stands for position c when cand_pos is
    None, else for cand_pos[c] (-1 = absent).  With apply_range only positions
    inside the candidate range of query t take part.  Returns ids ascending.
    """
    scores = np.asarray(scores, dtype=np.float32)
    pos = np.arange(scores.shape[0], dtype=np.int64) if cand_pos is None \
        else np.asarray(cand_pos, dtype=np.int64)
    keep = pos >= 0
    if apply_range:
        lo, hi = candidate_range(t, S, W)
        keep &= (pos >= lo) & (pos <= hi)
    return top_k(scores[keep], pos[keep], k)


# ----------------------------------------------------------------------------
# attention (Eq. 3)
# ----------------------------------------------------------------------------


def attend(q, k, v, S_t, sm_scale):
    """Softmax attention of one query over the key/value rows listed in S_t.

    q [H, d_qk]; k [n, d_qk]; v [n, d_v] (for the MLA latent v is k[:, :d_v]);
    the same k/v row serves every head.  Returns (out [H, d_v], lse [H]) with
    lse = log sum_s exp(sm_scale * q.k_s).
    """
    q = np.asarray(q, dtype=np.float64)
    S_t = np.asarray(S_t, dtype=np.int64)
    ks = np.asarray(k)[S_t].astype(np.float64)     # gather first: the caches may be huge float32 arrays
    vs = np.asarray(v)[S_t].astype(np.float64)
    z = sm_scale * (q @ ks.T)                 # [H, |S_t|]
    m = z.max(axis=1, keepdims=True)
    e = np.exp(z - m)
    den = e.sum(axis=1, keepdims=True)
    out = (e / den) @ vs
    lse = (m + np.log(den))[:, 0]
    return out, lse


def merge_partials(outs, lses):
    """Combine attention results over disjoint key sets by their log-sum-exp.

    out = sum_i exp(lse_i - lse) * out_i,  lse = log sum_i exp(lse_i).
    (The rescaling merge of the two-branch operator, Sec. 4.1.1, and of the
    sharded-cache decode, App. B.)
    """
    lses = np.stack([np.asarray(l, dtype=np.float64) for l in lses])     # [n, H]
    m = lses.max(axis=0)
    lse = m + np.log(np.exp(lses - m).sum(axis=0))
    out = sum(np.exp(l - lse)[:, None] * np.asarray(o, dtype=np.float64) for o, l in zip(outs, lses))
    return out, lse


# ----------------------------------------------------------------------------
# paged caches (App. B: caches are held as pages)
# ----------------------------------------------------------------------------


def paged_rows(positions, page_table_row, kv_page):
    """Logical positions of one sequence -> physical row numbers in the pool.

    The pool is [n_phys_pages, kv_page, d] seen as rows; logical page i of the
    sequence lives in physical page page_table_row[i].
    """
    positions = np.asarray(positions, dtype=np.int64)
    pt = np.asarray(page_table_row, dtype=np.int64)
    return pt[positions // kv_page] * kv_page + positions % kv_page


def gather_paged(pool_rows, page_table_row, n, kv_page):
    """The first n logical rows of one sequence, read through its page table."""
    return np.asarray(pool_rows)[paged_rows(np.arange(n), page_table_row, kv_page)]


# ----------------------------------------------------------------------------
# whole path for one query
# ----------------------------------------------------------------------------


def layer_group_query(t, q_I, w, k_hat, km, q_layers, k_layers, v_layers, *, P, B, M, Ksp, S, W,
                      sm_scale, hi_enable=True):
    """Indexer once, attention in each of the R layers of the group with the same set.

    q_layers[r] [H, d_qk], k_layers[r] [n, d_qk], v_layers[r] [n, d_v].
    Returns (sparse, pages, [out_r], [lse_r]).
    """
    sparse, pages = select_sparse(t, q_I, w, k_hat, km, P=P, B=B, M=M, Ksp=Ksp, S=S, W=W,
                                  hi_enable=hi_enable)
    S_t = index_set(t, S, W, sparse)
    outs, lses = [], []
    for q, k, v in zip(q_layers, k_layers, v_layers):
        o, l = attend(q, k, v, S_t, sm_scale)
        outs.append(o)
        lses.append(l)
    return sparse, pages, outs, lses
