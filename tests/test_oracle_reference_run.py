"""Pins for oracle/reference_run.py (CPU only): the glue that applies the oracle to host copies of a workload.

Each check compares the glue with something written here independently of it: hand-counted set overlaps
(the Overlap of App. C), caches gathered by explicit Python loops over a page table, scalar-loop block means and a
scalar-loop softmax on a tiny problem whose value dimension is shorter than its key dimension.
"""
import math

import numpy as np

from oracle import lsa_oracle as orc
from oracle import reference_run as ref


# ---- Overlap (App. C): card(S_gpu & S_ref) / card(S_ref) -------------------------------------------------------

def test_overlap_on_hand_counted_sets():
    assert ref.overlap([1, 2, 3], [2, 3, 4]) == 2 / 3
    assert ref.overlap([2, 3, 4], [1, 2, 3]) == 2 / 3
    assert ref.overlap([], []) == 1.0
    assert ref.overlap([5], []) == 0.0          # something selected where nothing should be
    assert ref.overlap([], [5]) == 0.0
    assert ref.overlap([7, 8, 9], [7, 8, 9]) == 1.0
    assert ref.overlap([9, 7, 8], [7, 8, 9]) == 1.0    # order is irrelevant: sets
    assert ref.overlap([1, 2], [3, 4]) == 0.0
    # the denominator is the reference set, not the union and not the GPU set
    assert ref.overlap([1, 2, 3, 4], [1, 2]) == 1.0
    assert ref.overlap([1], [1, 2, 3, 4]) == 0.25
    # numpy inputs with a -1 pad cut off by the caller behave like lists
    assert ref.overlap(np.array([4, 6, 10], dtype=np.int32), np.array([4, 10, 11, 12], dtype=np.int64)) == 0.5


def test_overlap_is_not_constant():
    """An overlap that always returned 1 would turn every selection check green: random sets, counted by loops."""
    rng = np.random.default_rng(0)
    seen = set()
    for _ in range(50):
        a = rng.choice(40, size=int(rng.integers(1, 20)), replace=False)
        b = rng.choice(40, size=int(rng.integers(1, 20)), replace=False)
        common = 0
        for x in b:
            for y in a:
                if x == y:
                    common += 1
        want = common / len(b)
        assert abs(ref.overlap(a, b) - want) < 1e-15
        seen.add(round(want, 6))
    assert len(seen) > 5


# ---- HostCaches ----------------------------------------------------------------------------------------------

def _tiny_caches(rng, n, d_i, d_qk, R, fp8):
    k_real = rng.standard_normal((n, d_i)) / math.sqrt(d_i)
    if fp8:
        codes = np.zeros((n, d_i), dtype=np.uint8)
        scale = np.zeros(n, dtype=np.float32)
        for s in range(n):
            codes[s], scale[s] = orc.quantize_token(k_real[s])
        k_idx = codes
    else:
        k_idx, scale = orc.bf16_round(k_real), None
    kv = [orc.bf16_round(rng.standard_normal((n, d_qk))) for _ in range(R)]
    return k_idx, scale, kv


def _mean_loops(k_hat, B):
    n, d = k_hat.shape
    nb = (n + B - 1) // B
    out = np.zeros((nb, d))
    for b in range(nb):
        cnt = 0
        for s in range(b * B, min(n, b * B + B)):
            out[b] += k_hat[s]
            cnt += 1
        out[b] /= cnt
    return orc.bf16_round(out)


def test_host_caches_contiguous_fields():
    rng = np.random.default_rng(1)
    n, d_i, d_qk, R, B = 45, 8, 12, 2, 4
    for fp8 in (False, True):
        k_idx, scale, kv = _tiny_caches(rng, n + 7, d_i, d_qk, R, fp8)    # pool longer than the sequence
        c = ref.HostCaches(k_idx, scale, kv, kv, B, n_key=n)
        assert c.k_hat.shape == (n, d_i) and c.k_hat.dtype == np.float64
        if fp8:
            # dequantised by hand: table value of the code times the token's scale
            table = orc.e4m3_decode(np.arange(256, dtype=np.uint8))
            for s in (0, 13, n - 1):
                for j in range(d_i):
                    assert c.k_hat[s, j] == table[k_idx[s, j]] * float(scale[s])
        else:
            assert np.array_equal(c.k_hat, k_idx[:n])
        # the mean cache uses the sub-block size handed in (not the page size, not 1), over the first n tokens only
        assert c.B == B
        assert np.array_equal(c.km, _mean_loops(c.k_hat, B))
        assert c.km.shape[0] == (n + B - 1) // B
        for r in range(R):
            assert np.array_equal(c.k[r], kv[r][:n]) and np.array_equal(c.v[r], kv[r][:n])
        kmax, kmin = c.minmax()
        for b in (0, c.km.shape[0] - 1):
            blk = c.k_hat[b * B:min(n, b * B + B)]
            assert np.all(kmax[b] >= blk.max(axis=0) - 1e-2) and np.all(kmin[b] <= blk.min(axis=0) + 1e-2)


def test_host_caches_paged_equal_unpaged():
    """A shuffled page table over pools gives the same logical caches as the contiguous arrays."""
    rng = np.random.default_rng(2)
    n, d_i, d_qk, R, B, page = 77, 8, 12, 2, 4, 16
    k_idx, scale, kv = _tiny_caches(rng, n, d_i, d_qk, R, fp8=True)
    n_pages = (n + page - 1) // page
    n_phys = n_pages + 3
    table = rng.permutation(n_phys)[:n_pages]
    # pools written by explicit loops: logical position s lives in physical row table[s // page] * page + s % page;
    # every other row holds junk that must never be read
    k_pool = rng.integers(0, 120, size=(n_phys * page, d_i)).astype(np.uint8)
    s_pool = rng.uniform(5.0, 6.0, size=n_phys * page).astype(np.float32)
    kv_pool = [rng.standard_normal((n_phys * page, d_qk)) * 50 for _ in range(R)]
    for s in range(n):
        row = int(table[s // page]) * page + s % page
        k_pool[row] = k_idx[s]
        s_pool[row] = scale[s]
        for r in range(R):
            kv_pool[r][row] = kv[r][s]
    flat = ref.HostCaches(k_idx, scale, kv, kv, B, n_key=n)
    paged = ref.HostCaches(k_pool, s_pool, kv_pool, kv_pool, B, n_key=n, page_table_row=table, kv_page=page)
    assert np.array_equal(paged.k_hat, flat.k_hat)
    assert np.array_equal(paged.km, flat.km)
    for r in range(R):
        assert np.array_equal(paged.k[r], flat.k[r]) and np.array_equal(paged.v[r], flat.v[r])
    a, b = paged.minmax(), flat.minmax()
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ---- select_query / attend_query ---------------------------------------------------------------------------

def _softmax_loops(q, k, v, rows, scale):
    """Eq. 3 with scalar loops: out[h] = sum_s softmax_s(scale q[h].k[s]) v[s] over the listed rows."""
    H, d_v = q.shape[0], v.shape[1]
    out = np.zeros((H, d_v))
    lse = np.zeros(H)
    for h in range(H):
        z = []
        for s in rows:
            dot = 0.0
            for c in range(q.shape[1]):
                dot += q[h, c] * k[s, c]
            z.append(scale * dot)
        m = max(z)
        den = sum(math.exp(x - m) for x in z)
        for x, s in zip(z, rows):
            p = math.exp(x - m) / den
            for c in range(d_v):
                out[h, c] += p * v[s, c]
        lse[h] = m + math.log(den)
    return out, lse


def test_select_query_equals_direct_oracle_call():
    rng = np.random.default_rng(3)
    n, H, d_i, B, P, M, Ksp, S, W = 200, 3, 8, 4, 16, 3, 20, 2, 24
    k_idx, scale, kv = _tiny_caches(rng, n, d_i, 6, 1, fp8=True)
    caches = ref.HostCaches(k_idx, scale, kv, kv, B, n_key=n)
    q = (rng.standard_normal((n, H, d_i)) / math.sqrt(d_i)).astype(np.float32)
    w = (rng.standard_normal((n, H)) / math.sqrt(H)).astype(np.float32)
    kw = dict(P=P, B=B, M=M, Ksp=Ksp, S=S, W=W)
    k_hat = orc.dequant_keys(k_idx, scale)
    km = _mean_loops(k_hat, B)
    differ = 0
    for t in (0, S + W - 1, S + W, 90, 151, n - 1):
        for hi in (True, False):
            got_s, got_p = ref.select_query(t, q[t], w[t], caches, hi_enable=hi, **kw)
            want_s, want_p = orc.select_sparse(t, q[t].astype(np.float64), w[t].astype(np.float64), k_hat, km,
                                               hi_enable=hi, **kw)
            assert np.array_equal(got_s, want_s) and np.array_equal(got_p, want_p)
        a, _ = ref.select_query(t, q[t], w[t], caches, hi_enable=True, **kw)
        b, _ = ref.select_query(t, q[t], w[t], caches, hi_enable=False, **kw)
        differ += int(not np.array_equal(a, b))
        # MinMax pooling reaches the oracle's Eq. 13 branch
        c, pc = ref.select_query(t, q[t], w[t], caches, pooling="minmax", **kw)
        d, pd = orc.select_sparse(t, q[t].astype(np.float64), w[t].astype(np.float64), k_hat, km,
                                  minmax=orc.block_minmax(k_hat, B), **kw)
        assert np.array_equal(c, d) and np.array_equal(pc, pd)
    assert differ > 0      # hi_enable is passed through: the binding budget M = 3 pages changes late queries


def test_attend_query_slices_the_value_and_builds_the_index_set():
    """d_v < d_qk: the value is the first d_v dims of the row; the set is sink + sparse + window (Eq. 6)."""
    rng = np.random.default_rng(4)
    n, H, d_qk, d_v, R, S, W = 60, 2, 6, 4, 2, 2, 5
    kv = [orc.bf16_round(rng.standard_normal((n, d_qk))) for _ in range(R)]
    caches = ref.HostCaches(orc.bf16_round(rng.standard_normal((n, 4))), None, kv, kv, 4, n_key=n)
    q = [rng.standard_normal((H, d_qk)).astype(np.float32) for _ in range(R)]
    scale = 0.37
    for t, sparse in ((40, [3, 9, 17, 30]), (3, []), (n - 1, [2, 50])):
        outs, lses = ref.attend_query(t, q, caches, np.array(sparse, dtype=np.int32), S=S, W=W, sm_scale=scale, d_v=d_v)
        rows = list(range(min(S, t + 1))) + list(sparse) + list(range(max(S, t - W + 1), t + 1))
        assert len(outs) == R and len(lses) == R
        for r in range(R):
            want_o, want_l = _softmax_loops(q[r].astype(np.float64), kv[r], kv[r][:, :d_v], rows, scale)
            assert outs[r].shape == (H, d_v)
            assert np.abs(outs[r] - want_o).max() < 1e-12
            assert np.abs(lses[r] - want_l).max() < 1e-12
    # layers are not mixed up: layer 1's output differs from layer 0's
    outs, _ = ref.attend_query(40, q, caches, np.array([3, 9]), S=S, W=W, sm_scale=scale, d_v=d_v)
    assert np.abs(outs[0] - outs[1]).max() > 1e-3
