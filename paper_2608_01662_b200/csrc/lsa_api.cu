// C ABI of liblsa: argument checking, workspace carving and the sequencing of the kernels.
// Every step of the path runs in the CUDA kernels of lsa_index.cu / lsa_attn.cu; nothing here
// computes on the host.
#include "../../include/lsa.h"

#include <cstdio>
#include <cstring>
#include <new>

#include "lsa_internal.h"

struct lsa_ctx {
  int device;
  cudaStream_t stream;
  uint8_t* ws;
  size_t ws_bytes;
  int sm_count;
  int64_t launches;
  char cuda_msg[256];
  // lsa_layer_group_host only
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in[2], ev_done[2], ev_out[2];
  // per-kernel timing (lsa_profile_*): event pairs recorded around the launches of each kernel class
  int tune[LSA_TUNE_COUNT];
  // Row lists of the last kernel launched through this context, if that kernel was a paged attention launch: the next
  // attention launch on the same lists may read them ahead of its programmatic dependency wait (the lists were
  // complete before that last kernel started).  Any other launch through the context clears it.
  const void* last_attn_rows;
  int prof_on;
  int prof_n;
  cudaEvent_t* prof_ev;   // 2 * kProfPairs events, created on first enable
  int* prof_cat;
};

namespace {

constexpr size_t kStatusBytes = 256;
constexpr int kMaxSplit = 16;
constexpr int kProfPairs = 4096;
constexpr int64_t kFusedBudget = 4096;        // candidate tokens per query the fused fine kernels keep in shared memory
constexpr int64_t kMaxBudget = 262144;        // largest recall budget M * P of the large-budget path
constexpr int64_t kFlatFusedMaxKeys = 4096;   // caches up to this length: the fused fine kernel scores every eligible page

// Runs `launch` (a callable returning cudaError_t), bracketed by an event pair of class `cat` when
// profiling is on and pairs are left.
template <class F>
cudaError_t timed(lsa_ctx* c, int cat, F launch) {
  const bool rec = c->prof_on && c->prof_ev != nullptr && c->prof_n < kProfPairs;
  if (cat != LSA_K_ATTN) c->last_attn_rows = nullptr;
  if (rec) cudaEventRecord(c->prof_ev[2 * c->prof_n], c->stream);
  const cudaError_t e = launch();
  if (rec) {
    cudaEventRecord(c->prof_ev[2 * c->prof_n + 1], c->stream);
    c->prof_cat[c->prof_n++] = cat;
  }
  return e;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int cuda_fail(lsa_ctx* c, cudaError_t e) {
  if (c) std::snprintf(c->cuda_msg, sizeof(c->cuda_msg), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
  return LSA_ERR_CUDA;
}

bool pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_params(const lsa_params* p, bool need_index, bool need_attn) {
  if (p == nullptr || p->struct_size != sizeof(lsa_params)) return LSA_ERR_ARG;
  if (p->k_sink < 0 || p->k_swa < 0 || p->k_sparse < 0) return LSA_ERR_ARG;
  if (p->paged != 0 && p->paged != 1) return LSA_ERR_ARG;
  if (need_index) {
    if (p->key_dtype != LSA_KEY_BF16 && p->key_dtype != LSA_KEY_E4M3) return LSA_ERR_ARG;
    if (p->page <= 0 || p->sub_block <= 0 || p->keep_pages <= 0) return LSA_ERR_ARG;
    if (!lsa::index_shape_supported(p->n_heads_idx, p->d_idx)) return LSA_ERR_SHAPE;
    if (p->page != 64 && p->page != 128 && p->page != 256) return LSA_ERR_SHAPE;
    if (p->page % p->sub_block != 0) return LSA_ERR_SHAPE;
    const int spp = p->page / p->sub_block;
    if (spp != 8 && spp != 16 && spp != 32) return LSA_ERR_SHAPE;
    const int64_t budget = static_cast<int64_t>(p->keep_pages) * p->page;
    if (budget > kFusedBudget) {
      // larger recall budgets: contiguous caches and the 64-head, 128-dim indexer only (scores go through the workspace)
      if (p->paged || p->n_heads_idx != 64 || p->d_idx != 128 || budget > kMaxBudget || budget % 128 != 0) return LSA_ERR_SHAPE;
    }
    if (p->k_sparse > 4096 || p->k_sparse % 4 != 0) return LSA_ERR_SHAPE;
    if (p->paged && p->kv_page != p->page) return LSA_ERR_SHAPE;
    if (p->pooling != LSA_POOL_MEAN && p->pooling != LSA_POOL_MINMAX) return LSA_ERR_ARG;
    if (p->pooling == LSA_POOL_MINMAX && p->paged) return LSA_ERR_SHAPE;   // the variant is built for contiguous caches
  }
  if (need_attn) {
    if (!lsa::attn_shape_supported(p->n_heads, p->d_qk, p->d_v)) return LSA_ERR_SHAPE;
    if (!(p->sm_scale > 0.f)) return LSA_ERR_ARG;
    if (p->paged && !pow2(p->kv_page)) return LSA_ERR_SHAPE;
  }
  return LSA_OK;
}

}  // namespace

int lsa::check_index_call(const lsa_params* p, const void* q_idx, const float* w, const void* k_idx, const float* k_scale,
                          const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key, const int32_t* page_table,
                          int64_t page_table_stride, const int32_t* ctx_len, int batch, const int32_t* sparse_idx,
                          const int32_t* n_sparse) {
  const int r = check_params(p, true, false);
  if (r != LSA_OK) return r;
  if (q_idx == nullptr || w == nullptr || k_idx == nullptr || sparse_idx == nullptr || n_sparse == nullptr) return LSA_ERR_ARG;
  if (p->hi_enable && kmean == nullptr) return LSA_ERR_ARG;
  if (p->key_dtype == LSA_KEY_E4M3 && k_scale == nullptr) return LSA_ERR_ARG;
  if (n_query < 0 || n_key < 0 || q_pos0 < 0) return LSA_ERR_ARG;
  if (p->paged) {
    if (page_table == nullptr || ctx_len == nullptr || batch <= 0 || page_table_stride <= 0) return LSA_ERR_ARG;
  } else if (q_pos0 + n_query > n_key) {
    return LSA_ERR_ARG;
  }
  if (!aligned16(q_idx) || !aligned16(w) || !aligned16(k_idx) || (kmean && !aligned16(kmean))) return LSA_ERR_SHAPE;
  return LSA_OK;
}

namespace {

// Workspace map.  All offsets are multiples of 256 bytes.
struct WsLayout {
  size_t page_scores, rows, n_rows, part_out, part_lse, fine_keys, fine_pages, wide_keys, total;
  size_t big_pages, big_np, big_keys;   // large recall budget (M * P > 4096): page lists and the candidates' keys
  int ps_ld, rows_ld;
};

// The page-score matrix comes last, so that the offsets of the other pieces do not depend on the cache length.
WsLayout ws_layout(const lsa_params* p, int64_t n_query, int64_t n_key_max, int batch) {
  WsLayout l{};
  size_t off = kStatusBytes;
  const int64_t nq = p->paged ? batch : n_query;
  l.rows_ld = p->k_sink + p->k_sparse + p->k_swa;
  if (p->paged) {
    l.rows = off;
    off += align_up(static_cast<size_t>(batch) * l.rows_ld * sizeof(int32_t), 256);
    l.n_rows = off;
    off += align_up(static_cast<size_t>(batch) * sizeof(int32_t), 256);
    l.part_out = off;
    off += align_up(static_cast<size_t>(batch) * kMaxSplit * p->n_heads * p->d_v * sizeof(float), 256);
    l.part_lse = off;
    off += align_up(static_cast<size_t>(batch) * kMaxSplit * p->n_heads * sizeof(float), 256);
    l.fine_keys = off;
    off += align_up(static_cast<size_t>(batch) * 4096 * sizeof(uint32_t), 256);
    l.fine_pages = off;
    off += align_up(static_cast<size_t>(batch) * 65 * sizeof(int32_t), 256);
  }
  const bool flat = !p->hi_enable && n_key_max > kFlatFusedMaxKeys;
  const bool tc_fine = !p->paged && p->n_heads_idx == 64 && p->d_idx == 128;
  if (!p->paged && (flat || tc_fine) && p->key_dtype == LSA_KEY_E4M3) {
    // e4m3 codes widened to bf16 once per call: dense scoring of the flat indexer, TMA source of the fine stage
    l.wide_keys = off;
    off += align_up(static_cast<size_t>(n_key_max) * p->d_idx * 2, 256);
  }
  const int64_t budget = static_cast<int64_t>(p->keep_pages) * p->page;
  if (!flat && !p->paged && budget > kFusedBudget) {
    l.big_pages = off;
    off += align_up(static_cast<size_t>(nq) * p->keep_pages * sizeof(int32_t), 256);
    l.big_np = off;
    off += align_up(static_cast<size_t>(nq) * sizeof(int32_t), 256);
    l.big_keys = off;
    off += align_up(static_cast<size_t>(nq) * budget * sizeof(uint32_t), 256);
  }
  const int P = p->page > 0 ? p->page : 64;
  // hierarchical: one score per page; flat: one score per token
  l.ps_ld = static_cast<int>(align_up(static_cast<size_t>(flat ? n_key_max : (n_key_max + P - 1) / P), 4));
  l.page_scores = off;
  off += align_up(static_cast<size_t>(nq) * l.ps_ld * sizeof(float), 256);
  l.total = off;
  return l;
}

int* status_word(lsa_ctx* c) { return c->ws ? reinterpret_cast<int*>(c->ws) : nullptr; }

// Number of row splits per sequence in paged (decode) attention.  Blocks run one per SM in waves; a block costs its
// share of the 64-key units plus a fixed part (Q load, tensor-memory set-up, fp32 partial output), taken as six
// units' worth.  The split count with the smallest estimate wins; ties go to fewer splits (less merging).  The
// tcgen05 kernel merges its splits inside a thread-block cluster and takes only the counts that allows.
int pick_split(int sm_count, int batch, int max_rows, bool tc_kernel) {
  const int units = (max_rows + 63) / 64;
  int best = 1;
  long best_cost = -1;
  for (int s = 1; s <= kMaxSplit && s <= units; ++s) {
    if (tc_kernel && !lsa::attn_tc_split_ok(s)) continue;
    const long waves = (static_cast<long>(batch) * s + sm_count - 1) / sm_count;
    const long cost = waves * ((units + s - 1) / s + 6);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

int run_index(lsa_ctx* c, const lsa_params* p, const void* q_idx, const float* w, const void* k_idx,
              const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key,
              const int32_t* page_table, int64_t pt_stride, const int32_t* ctx_len, int batch,
              int32_t* sparse_idx, int32_t* n_sparse, int32_t* pages_out, int32_t* rows_out = nullptr,
              int32_t* n_rows_out = nullptr) {
  const int64_t nq = p->paged ? batch : n_query;
  if (nq == 0) return LSA_OK;
  const int64_t n_key_max = p->paged ? pt_stride * p->kv_page : n_key;
  const bool flat = !p->hi_enable && n_key_max > kFlatFusedMaxKeys;
  const int64_t chunk = (!p->paged && p->q_chunk > 0) ? p->q_chunk : nq;
  const WsLayout l = ws_layout(p, chunk < nq ? chunk : nq, n_key_max, batch);
  if (c->ws == nullptr || l.total > c->ws_bytes) return LSA_ERR_WORKSPACE;
  for (int64_t q0 = 0; q0 < nq; q0 += chunk) {
    const int64_t n = nq - q0 < chunk ? nq - q0 : chunk;
    lsa::IndexArgs a{};
    a.HI = p->n_heads_idx; a.DI = p->d_idx; a.key_e4m3 = p->key_dtype == LSA_KEY_E4M3;
    a.P = p->page; a.B = p->sub_block; a.M = p->keep_pages; a.Ksp = p->k_sparse; a.S = p->k_sink; a.W = p->k_swa;
    a.hi_enable = p->hi_enable; a.paged = p->paged;
    a.q_idx = static_cast<const uint8_t*>(q_idx) + q0 * p->n_heads_idx * p->d_idx * 2;
    a.w = w + q0 * p->n_heads_idx;
    a.k_idx = k_idx; a.k_scale = k_scale; a.kmean = kmean;
    a.q_pos0 = q_pos0 + q0; a.n_query = static_cast<int>(n); a.n_key = n_key;
    a.page_table = page_table; a.pt_stride = pt_stride; a.ctx_len = ctx_len;
    a.page_scores = reinterpret_cast<float*>(c->ws + l.page_scores); a.ps_ld = l.ps_ld;
    a.sparse_idx = sparse_idx + q0 * p->k_sparse; a.n_sparse = n_sparse + q0;
    a.pages_out = pages_out ? pages_out + q0 * p->keep_pages : nullptr;
    a.rows_out = p->paged ? rows_out : nullptr;   // a5 fused into the last selection kernel (decode)
    a.n_rows_out = n_rows_out;
    a.status = status_word(c);
    a.fine_parts = 1;
    a.sm_count = c->sm_count;
    const bool paged_tc = p->paged && lsa::paged_scores_tc_supported(a);   // token scores of cache pages on tcgen05
    if (flat && p->paged && !paged_tc) return LSA_ERR_SHAPE;   // the flat indexer over long paged caches needs that kernel
    if (p->paged && !flat && c->tune[LSA_TUNE_FINE_PAGED_TC] == 0 && lsa::fine_paged_tc_supported(a)) {
      a.fine_cluster = 1;
      a.fine_parts = 2;   // (the kernel writes the cache rows itself)
    } else if (paged_tc && (flat || c->tune[LSA_TUNE_FINE_PAGED_TC] == 1)) {
      a.fine_paged_tc = 1;
      a.fine_parts = 2;   // (marks the split path: the top-K kernel writes the cache rows itself)
      a.fine_keys = reinterpret_cast<uint32_t*>(c->ws + l.fine_keys);
      a.fine_pages = reinterpret_cast<int32_t*>(c->ws + l.fine_pages);
    } else if (p->paged) {
      // few queries and many SMs: several blocks score each query's candidates, a second kernel selects
      int parts = 2 * c->sm_count / (batch > 0 ? batch : 1);   // two scoring blocks fit one SM
      parts = parts > 4 ? 4 : parts;
      if (parts > 1) {
        a.fine_parts = parts;
        a.fine_keys = reinterpret_cast<uint32_t*>(c->ws + l.fine_keys);
        a.fine_pages = reinterpret_cast<int32_t*>(c->ws + l.fine_pages);
      }
    }
    cudaError_t e = cudaSuccess;
    if (!flat && a.key_e4m3 && l.wide_keys != 0) {
      // the fine stage reads key tiles by TMA from a bf16 copy of the codes (exact; scales enter after the dot products)
      void* wide = c->ws + l.wide_keys;
      if (q0 == 0) e = timed(c, LSA_K_MEANS, [&] { return lsa::launch_widen_e4m3(k_idx, wide, n_key * p->d_idx, c->stream, &c->launches); });
      if (e != cudaSuccess) return cuda_fail(c, e);
      a.k_wide = wide;
    }
    if (flat && p->paged) {
      // Eq. 7 without the hierarchy over paged caches: token scores of every page of the scoring range (per-token
      // scale applied), the top-K_sparse of each sequence's row, then the cache rows.
      e = timed(c, LSA_K_COARSE, [&] { return lsa::launch_paged_scores_tc(a, 1, c->sm_count, c->stream, &c->launches); });
      if (e == cudaSuccess)
        e = timed(c, LSA_K_SELECT, [&] {
          return lsa::launch_select(a.page_scores, a.ps_ld, nullptr, nullptr, 0, a.n_query, n_key_max, p->k_sparse, 1, p->k_sink,
                                    p->k_swa, a.sparse_idx, a.n_sparse, c->stream, &c->launches, ctx_len);
        });
      if (e == cudaSuccess && a.rows_out != nullptr)
        e = timed(c, LSA_K_CONVERT, [&] {
          return lsa::launch_convert(p->k_sink, p->k_swa, p->k_sparse, p->paged, p->kv_page, a.sparse_idx, a.n_sparse, a.q_pos0,
                                     a.n_query, page_table, pt_stride, ctx_len, a.rows_out, a.n_rows_out, nullptr, c->stream,
                                     &c->launches);
        });
      if (e == cudaSuccess && a.pages_out != nullptr)
        e = cudaMemsetAsync(a.pages_out, 0xff, static_cast<size_t>(a.n_query) * p->keep_pages * sizeof(int32_t), c->stream);
      if (e != cudaSuccess) return cuda_fail(c, e);
      continue;
    }
    if (flat) {
      // Eq. 7 without the hierarchy: dense causal token scores (the coarse kernel with one token per "page"), then
      // the top-K_sparse of each row.  e4m3 keys are widened to bf16 once; their scale enters at the comparison.
      const void* keys_bf16 = k_idx;
      if (a.key_e4m3) {
        void* wide = c->ws + l.wide_keys;
        if (q0 == 0) e = timed(c, LSA_K_MEANS, [&] { return lsa::launch_widen_e4m3(k_idx, wide, n_key * p->d_idx, c->stream, &c->launches); });
        keys_bf16 = wide;
      }
      lsa::IndexArgs d = a;
      d.P = 1; d.B = 1; d.M = 0; d.kmean = keys_bf16; d.hi_enable = 1;
      if (e == cudaSuccess)
        e = timed(c, LSA_K_COARSE, [&] { return lsa::launch_coarse_best(d, c->tune[LSA_TUNE_COARSE_GROUPS], c->stream, &c->launches); });
      if (e == cudaSuccess)
        e = timed(c, LSA_K_SELECT, [&] {
          return lsa::launch_select(a.page_scores, a.ps_ld, nullptr, a.key_e4m3 ? k_scale : nullptr, a.q_pos0, a.n_query,
                                    n_key, p->k_sparse, 1, p->k_sink, p->k_swa, a.sparse_idx, a.n_sparse, c->stream,
                                    &c->launches);
        });
      if (e == cudaSuccess && a.pages_out != nullptr)
        e = cudaMemsetAsync(a.pages_out, 0xff, static_cast<size_t>(a.n_query) * p->keep_pages * sizeof(int32_t), c->stream);
      if (e != cudaSuccess) return cuda_fail(c, e);
      continue;
    }
    if (p->hi_enable && p->pooling == LSA_POOL_MINMAX)
      e = timed(c, LSA_K_COARSE, [&] { return lsa::launch_coarse_minmax(a, c->stream, &c->launches); });
    else if (p->hi_enable)
      e = timed(c, LSA_K_COARSE, [&] { return lsa::launch_coarse_best(a, c->tune[LSA_TUNE_COARSE_GROUPS], c->stream, &c->launches); });
    if (e == cudaSuccess && l.big_keys != 0) {
      // recall budget beyond one block's shared memory: page lists, fine scores through the workspace, top-K over them
      if (!lsa::fine_big_supported(a)) return LSA_ERR_SHAPE;
      e = timed(c, LSA_K_FINE_SELECT, [&] {
        return lsa::launch_fine_big(a, reinterpret_cast<int32_t*>(c->ws + l.big_pages), reinterpret_cast<int32_t*>(c->ws + l.big_np),
                                    reinterpret_cast<uint32_t*>(c->ws + l.big_keys), c->stream, &c->launches);
      });
      if (e != cudaSuccess) return cuda_fail(c, e);
      continue;
    }
    if (e == cudaSuccess) e = timed(c, LSA_K_FINE_SELECT, [&] { return lsa::launch_fine_select(a, c->stream, &c->launches); });
    if (e == cudaSuccess && a.rows_out != nullptr && a.fine_parts <= 1)
      // only the split fine stage writes the cache rows itself (in its top-K kernel)
      e = timed(c, LSA_K_CONVERT, [&] {
        return lsa::launch_convert(p->k_sink, p->k_swa, p->k_sparse, p->paged, p->kv_page, a.sparse_idx, a.n_sparse, a.q_pos0,
                                   a.n_query, page_table, pt_stride, ctx_len, a.rows_out, a.n_rows_out, nullptr, c->stream,
                                   &c->launches);
      });
    if (e != cudaSuccess) return cuda_fail(c, e);
  }
  return LSA_OK;
}

int run_attn(lsa_ctx* c, const lsa_params* p, const void* q, const void* k, const void* v, int64_t ld_k,
             int64_t ld_v, const int32_t* sparse_idx, const int32_t* n_sparse, const int32_t* rows,
             const int32_t* n_rows, int64_t q_pos0, int64_t n_query, const int32_t* ctx_len, int batch,
             void* out, float* lse, int64_t n_key = 0) {
  const int64_t nq = p->paged ? batch : n_query;
  if (nq == 0) return LSA_OK;
  lsa::AttnArgs a{};
  a.H = p->n_heads; a.DQK = p->d_qk; a.DV = p->d_v; a.S = p->k_sink; a.W = p->k_swa; a.Ksp = p->k_sparse;
  a.paged = p->paged; a.sm_scale = p->sm_scale;
  a.q = q; a.k = k; a.v = v; a.ld_k = ld_k; a.ld_v = ld_v;
  a.sparse_idx = sparse_idx; a.n_sparse = n_sparse; a.rows = rows; a.n_rows = n_rows;
  a.rows_ld = p->k_sink + p->k_sparse + p->k_swa;
  a.n_key = p->paged ? 0 : n_key;   // (the checking build validates caller-given row numbers against it)
  a.q_pos0 = q_pos0; a.n_query = static_cast<int>(nq); a.ctx_len = ctx_len; a.out = out; a.lse = lse;
  a.n_split = 1; a.status = status_word(c);
  a.qk_waits_pv = c->tune[LSA_TUNE_ATTN_PV_WAIT];
  a.pv_issuers = p->paged ? 4 : 2;   // decode waits on HBM gathers, prefill on the tensor pipe
  a.gather4 = c->tune[LSA_TUNE_ATTN_GATHER];
  a.rows_stable = rows != nullptr && c->last_attn_rows == rows;
  const bool use_tc = c->tune[LSA_TUNE_ATTN_TC] && lsa::attn_tc_supported(a);
  if (p->paged) {
    const WsLayout l = ws_layout(p, nq, 0, batch);
    if (c->ws == nullptr || l.total > c->ws_bytes) return LSA_ERR_WORKSPACE;
    a.n_split = c->tune[LSA_TUNE_ATTN_SPLIT] > 0 ? c->tune[LSA_TUNE_ATTN_SPLIT]
                                                 : pick_split(c->sm_count, batch, a.rows_ld, use_tc);
    if (use_tc && !lsa::attn_tc_split_ok(a.n_split)) return LSA_ERR_ARG;
    a.part_out = reinterpret_cast<float*>(c->ws + l.part_out);
    a.part_lse = reinterpret_cast<float*>(c->ws + l.part_lse);
  }
  if (a.H == 64 && !(v == k && ld_v == ld_k)) return LSA_ERR_SHAPE;
  cudaError_t e = timed(c, LSA_K_ATTN, [&] {
    return use_tc ? lsa::launch_attn_tc(a, c->stream, &c->launches) : lsa::launch_attn(a, c->stream, &c->launches);
  });
  c->last_attn_rows = (e == cudaSuccess && use_tc && p->paged) ? rows : nullptr;
  if (e == cudaSuccess && a.n_split > 1 && !use_tc) e = timed(c, LSA_K_MERGE, [&] { return lsa::launch_merge(a, c->stream, &c->launches); });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

}  // namespace

extern "C" {

int lsa_create(lsa_ctx** ctx, int device, void* cuda_stream, void* workspace, size_t workspace_bytes) {
  if (ctx == nullptr) return LSA_ERR_ARG;
  *ctx = nullptr;
  if (workspace != nullptr && (reinterpret_cast<uintptr_t>(workspace) & 255u)) return LSA_ERR_ARG;
  if (workspace != nullptr && workspace_bytes < kStatusBytes) return LSA_ERR_WORKSPACE;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return LSA_ERR_CUDA;
  lsa_ctx* c = new (std::nothrow) lsa_ctx();
  if (c == nullptr) return LSA_ERR_ARG;
  std::memset(c, 0, sizeof(*c));
  c->device = device;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->ws = static_cast<uint8_t*>(workspace);
  c->ws_bytes = workspace ? workspace_bytes : 0;
  c->tune[LSA_TUNE_COARSE_GROUPS] = 2;
  c->tune[LSA_TUNE_ATTN_TC] = 1;
  c->tune[LSA_TUNE_ATTN_GATHER] = 0;   // measured: the TMA unit paces four-row gathers below what 16-byte cp.async reaches
  e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming);
  }
  if (e == cudaSuccess && c->ws) e = cudaMemsetAsync(c->ws, 0, kStatusBytes, c->stream);
  if (e != cudaSuccess) {
    delete c;
    return LSA_ERR_CUDA;
  }
  *ctx = c;
  return LSA_OK;
}

int lsa_destroy(lsa_ctx* c) {
  if (c == nullptr) return LSA_ERR_ARG;
  cudaSetDevice(c->device);
  for (int i = 0; i < 2; ++i) {
    if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
    if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
    if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
  }
  if (c->prof_ev) {
    for (int i = 0; i < 2 * kProfPairs; ++i) cudaEventDestroy(c->prof_ev[i]);
    delete[] c->prof_ev;
    delete[] c->prof_cat;
  }
  if (c->copy_in) cudaStreamDestroy(c->copy_in);
  if (c->copy_out) cudaStreamDestroy(c->copy_out);
  delete c;
  return LSA_OK;
}

int lsa_workspace_bytes(const lsa_params* p, int64_t n_query, int64_t n_key_max, int batch, size_t* bytes) {
  if (bytes == nullptr || n_query < 0 || n_key_max < 0 || batch < 0) return LSA_ERR_ARG;
  const int r = check_params(p, true, true);
  if (r != LSA_OK) return r;
  int64_t nq = n_query;
  if (!p->paged && p->q_chunk > 0 && p->q_chunk < nq) nq = p->q_chunk;
  *bytes = ws_layout(p, nq, n_key_max, batch).total;
  return LSA_OK;
}

int lsa_status(lsa_ctx* c, int* device_status) {
  if (c == nullptr || device_status == nullptr) return LSA_ERR_ARG;
  *device_status = 0;
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e);
  if (c->ws == nullptr) return LSA_OK;
  e = cudaMemcpyAsync(device_status, c->ws, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws, 0, sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

int lsa_selftest_wait(lsa_ctx* c, int64_t budget_cycles) {
  if (c == nullptr || budget_cycles < 0 || budget_cycles > (1ll << 31)) return LSA_ERR_ARG;
  if (c->ws == nullptr) return LSA_ERR_WORKSPACE;
  const cudaError_t e = lsa::launch_selftest_wait(status_word(c), budget_cycles, nullptr, c->stream, &c->launches);
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

const char* lsa_strerror(int err) {
  switch (err) {
    case LSA_OK: return "ok";
    case LSA_ERR_ARG: return "invalid argument";
    case LSA_ERR_SHAPE: return "unsupported shape or alignment";
    case LSA_ERR_WORKSPACE: return "workspace missing or too small";
    case LSA_ERR_CUDA: return "CUDA runtime error";
    case LSA_ERR_TIMEOUT: return "device-side wait timed out";
    case LSA_ERR_CAPACITY: return "request exceeds the fixed scratch capacity of this entry point";
    case LSA_ERR_INDEX: return "cache row number outside the cache (checking build)";
    default: return "unknown error";
  }
}

const char* lsa_last_cuda_error(lsa_ctx* c) { return c ? c->cuda_msg : ""; }

int lsa_tune(lsa_ctx* c, int knob, int value) {
  if (c == nullptr || knob < 0 || knob >= LSA_TUNE_COUNT) return LSA_ERR_ARG;
  if (knob == LSA_TUNE_COARSE_GROUPS && value != 1 && value != 2) return LSA_ERR_ARG;
  if (knob == LSA_TUNE_ATTN_SPLIT && (value < 0 || value > kMaxSplit)) return LSA_ERR_ARG;
  if (knob == LSA_TUNE_ATTN_PV_WAIT && value != 0 && value != 1) return LSA_ERR_ARG;
  if (knob == LSA_TUNE_ATTN_GATHER && value != 0 && value != 1) return LSA_ERR_ARG;
  if (knob == LSA_TUNE_FINE_PAGED_TC && (value < 0 || value > 2)) return LSA_ERR_ARG;
  c->tune[knob] = value;
  return LSA_OK;
}

int lsa_profile_enable(lsa_ctx* c, int on) {
  if (c == nullptr) return LSA_ERR_ARG;
  if (on && c->prof_ev == nullptr) {
    c->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfPairs];
    c->prof_cat = new (std::nothrow) int[kProfPairs];
    if (c->prof_ev == nullptr || c->prof_cat == nullptr) return LSA_ERR_ARG;
    for (int i = 0; i < 2 * kProfPairs; ++i) {
      const cudaError_t e = cudaEventCreate(&c->prof_ev[i]);
      if (e != cudaSuccess) return cuda_fail(c, e);
    }
  }
  c->prof_on = on ? 1 : 0;
  c->prof_n = 0;
  return LSA_OK;
}

int lsa_profile_read(lsa_ctx* c, double* total_ms, int64_t* launches) {
  if (c == nullptr || total_ms == nullptr || launches == nullptr) return LSA_ERR_ARG;
  for (int i = 0; i < LSA_K_COUNT; ++i) {
    total_ms[i] = 0.0;
    launches[i] = 0;
  }
  cudaError_t e = cudaStreamSynchronize(c->stream);
  for (int i = 0; i < c->prof_n && e == cudaSuccess; ++i) {
    float ms = 0.f;
    e = cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]);
    total_ms[c->prof_cat[i]] += ms;
    launches[c->prof_cat[i]] += 1;
  }
  c->prof_n = 0;
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}
int64_t lsa_launch_count(lsa_ctx* c) { return c ? c->launches : 0; }

int lsa_block_means(lsa_ctx* c, const lsa_params* p, const void* k_idx, const float* k_scale, int64_t n_key,
                    const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
                    void* kmean) {
  if (c == nullptr) return LSA_ERR_ARG;
  int r = check_params(p, true, false);
  if (r != LSA_OK) return r;
  if (k_idx == nullptr || kmean == nullptr || n_key < 0) return LSA_ERR_ARG;
  if (p->key_dtype == LSA_KEY_E4M3 && k_scale == nullptr) return LSA_ERR_ARG;
  if (p->paged && (page_table == nullptr || ctx_len == nullptr || batch <= 0 || page_table_stride <= 0)) return LSA_ERR_ARG;
  if (!aligned16(k_idx) || !aligned16(kmean)) return LSA_ERR_SHAPE;
  if (p->pooling == LSA_POOL_MINMAX) {
    const cudaError_t em = timed(c, LSA_K_MEANS, [&] {
      return lsa::launch_block_minmax(p->d_idx, p->key_dtype == LSA_KEY_E4M3, p->sub_block, k_idx, k_scale, n_key, kmean,
                                      c->stream, &c->launches);
    });
    return em == cudaSuccess ? LSA_OK : cuda_fail(c, em);
  }
  cudaError_t e = timed(c, LSA_K_MEANS, [&] {
    return lsa::launch_block_means(p->d_idx, p->key_dtype == LSA_KEY_E4M3, p->sub_block, p->kv_page, k_idx, k_scale,
                                   n_key, p->paged ? page_table : nullptr, page_table_stride, ctx_len, batch, kmean,
                                   c->stream, &c->launches);
  });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

int lsa_append(lsa_ctx* c, const lsa_params* p, const void* k_new, void* k_idx, float* k_scale, void* kmean,
               const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
               int32_t* ctx_len_out, int n_kv, const void* const* kv_new, void* const* kv_pool, int64_t kv_row_bytes) {
  if (c == nullptr) return LSA_ERR_ARG;
  int r = check_params(p, true, false);
  if (r != LSA_OK) return r;
  if (!p->paged || p->pooling != LSA_POOL_MEAN) return LSA_ERR_SHAPE;
  if (k_new == nullptr || k_idx == nullptr || kmean == nullptr || page_table == nullptr || ctx_len == nullptr) return LSA_ERR_ARG;
  if (batch < 0 || page_table_stride <= 0) return LSA_ERR_ARG;
  if (p->key_dtype == LSA_KEY_E4M3 && k_scale == nullptr) return LSA_ERR_ARG;
  if (n_kv < 0 || n_kv > 8) return LSA_ERR_ARG;
  if (n_kv > 0 && (kv_new == nullptr || kv_pool == nullptr || kv_row_bytes <= 0 || kv_row_bytes % 16 != 0)) return LSA_ERR_ARG;
  if (!aligned16(k_idx) || !aligned16(kmean) || !aligned16(k_new)) return LSA_ERR_SHAPE;
  lsa::AppendArgs a{};
  a.DI = p->d_idx; a.key_e4m3 = p->key_dtype == LSA_KEY_E4M3; a.B = p->sub_block; a.kv_page = p->kv_page;
  a.batch = batch; a.n_kv = n_kv;
  a.k_new = k_new; a.k_idx = k_idx; a.k_scale = k_scale; a.kmean = kmean;
  a.page_table = page_table; a.pt_stride = page_table_stride; a.ctx_len = ctx_len; a.ctx_len_out = ctx_len_out;
  for (int i = 0; i < n_kv; ++i) {
    if (kv_new[i] == nullptr || kv_pool[i] == nullptr || !aligned16(kv_new[i]) || !aligned16(kv_pool[i])) return LSA_ERR_ARG;
    a.kv_new[i] = kv_new[i];
    a.kv_pool[i] = kv_pool[i];
  }
  a.kv_row_bytes = kv_row_bytes;
  cudaError_t e = timed(c, LSA_K_MEANS, [&] { return lsa::launch_append(a, c->stream, &c->launches); });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

// lsa_index with its argument checks; rows_out / n_rows_out (paged caches): also write what lsa_convert would
static int index_checked(lsa_ctx* c, const lsa_params* p, const void* q_idx, const float* w, const void* k_idx,
                         const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key,
                         const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
                         int32_t* sparse_idx, int32_t* n_sparse, int32_t* pages_out, int32_t* rows_out,
                         int32_t* n_rows_out) {
  if (c == nullptr) return LSA_ERR_ARG;
  const int r = lsa::check_index_call(p, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, page_table,
                                      page_table_stride, ctx_len, batch, sparse_idx, n_sparse);
  if (r != LSA_OK) return r;
  return run_index(c, p, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, page_table, page_table_stride,
                   ctx_len, batch, sparse_idx, n_sparse, pages_out, rows_out, n_rows_out);
}

int lsa_index(lsa_ctx* c, const lsa_params* p, const void* q_idx, const float* w, const void* k_idx,
              const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key,
              const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
              int32_t* sparse_idx, int32_t* n_sparse, int32_t* pages_out) {
  return index_checked(c, p, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, page_table, page_table_stride,
                       ctx_len, batch, sparse_idx, n_sparse, pages_out, nullptr, nullptr);
}

int lsa_select(lsa_ctx* c, const lsa_params* p, const float* scores, int64_t ld_scores, const int32_t* cand_pos,
               int64_t q_pos0, int64_t n_query, int64_t n_cand, int32_t k, int32_t apply_range, int32_t* idx_out,
               int32_t* n_out) {
  if (c == nullptr || p == nullptr || p->struct_size != sizeof(lsa_params)) return LSA_ERR_ARG;
  if (scores == nullptr || idx_out == nullptr || n_out == nullptr) return LSA_ERR_ARG;
  if (n_query < 0 || n_cand < 0 || k < 0 || ld_scores < n_cand || q_pos0 < 0) return LSA_ERR_ARG;
  if (k > 8192 || n_cand > 0x7fffffff) return LSA_ERR_SHAPE;
  if (n_query == 0 || k == 0) return LSA_OK;
  cudaError_t e = timed(c, LSA_K_SELECT, [&] {
    return lsa::launch_select(scores, ld_scores, cand_pos, nullptr, q_pos0, static_cast<int>(n_query), n_cand, k, apply_range,
                              p->k_sink, p->k_swa, idx_out, n_out, c->stream, &c->launches);
  });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

int lsa_convert(lsa_ctx* c, const lsa_params* p, const int32_t* sparse_idx, const int32_t* n_sparse, int64_t q_pos0,
                int64_t n_query, const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len,
                int batch, int32_t* rows_out, int32_t* n_rows_out, int32_t* runs_out) {
  if (c == nullptr || p == nullptr || p->struct_size != sizeof(lsa_params)) return LSA_ERR_ARG;
  if (sparse_idx == nullptr || n_sparse == nullptr || rows_out == nullptr || n_rows_out == nullptr) return LSA_ERR_ARG;
  if (p->paged && (page_table == nullptr || ctx_len == nullptr || batch <= 0 || p->kv_page <= 0)) return LSA_ERR_ARG;
  const int64_t nq = p->paged ? batch : n_query;
  if (nq < 0 || q_pos0 < 0) return LSA_ERR_ARG;
  cudaError_t e = timed(c, LSA_K_CONVERT, [&] {
    return lsa::launch_convert(p->k_sink, p->k_swa, p->k_sparse, p->paged, p->kv_page, sparse_idx, n_sparse, q_pos0,
                               static_cast<int>(nq), page_table, page_table_stride, ctx_len, rows_out, n_rows_out,
                               runs_out, c->stream, &c->launches);
  });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

int lsa_sparse_attn(lsa_ctx* c, const lsa_params* p, const void* q, const void* k, const void* v, int64_t ld_k,
                    int64_t ld_v, const int32_t* sparse_idx, const int32_t* n_sparse, const int32_t* rows,
                    const int32_t* n_rows, int64_t q_pos0, int64_t n_query, int64_t n_key, const int32_t* ctx_len,
                    int batch, void* out, float* lse) {
  if (c == nullptr) return LSA_ERR_ARG;
  int r = check_params(p, false, true);
  if (r != LSA_OK) return r;
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return LSA_ERR_ARG;
  if (rows == nullptr && (sparse_idx == nullptr || n_sparse == nullptr)) return LSA_ERR_ARG;
  if (rows != nullptr && n_rows == nullptr) return LSA_ERR_ARG;
  if (p->paged && (rows == nullptr || ctx_len == nullptr || batch <= 0)) return LSA_ERR_ARG;
  if (n_query < 0 || q_pos0 < 0 || n_key < 0) return LSA_ERR_ARG;
  if (ld_k < p->d_qk || ld_v < p->d_v || (ld_k % 8) || (ld_v % 8)) return LSA_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return LSA_ERR_SHAPE;
  return run_attn(c, p, q, k, v, ld_k, ld_v, sparse_idx, n_sparse, rows, n_rows, q_pos0, n_query, ctx_len, batch, out, lse, n_key);
}

int lsa_merge(lsa_ctx* c, const lsa_params* p, int n_parts, const void* const* outs, const float* const* lses,
              int64_t n_query, void* out, float* lse) {
  if (c == nullptr || p == nullptr || p->struct_size != sizeof(lsa_params)) return LSA_ERR_ARG;
  if (n_parts < 1 || n_parts > 8 || outs == nullptr || lses == nullptr || out == nullptr || n_query < 0) return LSA_ERR_ARG;
  if (p->n_heads <= 0 || p->d_v <= 0 || (p->d_v % 2)) return LSA_ERR_SHAPE;
  lsa::MergeArgs a{};
  a.n_parts = n_parts; a.H = p->n_heads; a.DV = p->d_v; a.n_query = static_cast<int>(n_query);
  for (int i = 0; i < n_parts; ++i) {
    if (outs[i] == nullptr || lses[i] == nullptr) return LSA_ERR_ARG;
    a.outs[i] = outs[i];
    a.lses[i] = lses[i];
  }
  a.out = out; a.lse = lse;
  cudaError_t e = timed(c, LSA_K_MERGE, [&] { return lsa::launch_merge_parts(a, c->stream, &c->launches); });
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

int lsa_layer_group(lsa_ctx* c, const lsa_params* p, const void* q_idx, const float* w, const void* k_idx,
                    const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key,
                    const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
                    const void* const* q, const void* const* k, const void* const* v, int64_t ld_k, int64_t ld_v,
                    void* const* out, float* const* lse, int32_t* sparse_idx, int32_t* n_sparse) {
  if (c == nullptr) return LSA_ERR_ARG;
  int r = check_params(p, true, true);
  if (r != LSA_OK) return r;
  if (p->n_layers <= 0 || q == nullptr || k == nullptr || v == nullptr || out == nullptr) return LSA_ERR_ARG;
  for (int i = 0; i < p->n_layers; ++i)
    if (q[i] == nullptr || k[i] == nullptr || v[i] == nullptr || out[i] == nullptr) return LSA_ERR_ARG;
  // paged caches: the index -> cache-row conversion (a5) rides in the indexer's last kernel
  int32_t* rows = nullptr;
  int32_t* n_rows = nullptr;
  if (p->paged) {
    if (page_table_stride <= 0 || batch <= 0) return LSA_ERR_ARG;
    const WsLayout l = ws_layout(p, batch, page_table_stride * p->kv_page, batch);
    if (c->ws == nullptr || l.total > c->ws_bytes) return LSA_ERR_WORKSPACE;
    rows = reinterpret_cast<int32_t*>(c->ws + l.rows);
    n_rows = reinterpret_cast<int32_t*>(c->ws + l.n_rows);
  }
  r = index_checked(c, p, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, page_table, page_table_stride,
                    ctx_len, batch, sparse_idx, n_sparse, nullptr, rows, n_rows);
  if (r != LSA_OK) return r;
  // The layers run one after another on the stream: in a model the query of layer r + 1 is computed from the output of
  // layer r, so they are never launched side by side.
  for (int i = 0; i < p->n_layers; ++i) {
    r = lsa_sparse_attn(c, p, q[i], k[i], v[i], ld_k, ld_v, sparse_idx, n_sparse, rows, n_rows, q_pos0, n_query,
                        n_key, ctx_len, batch, out[i], lse ? lse[i] : nullptr);
    if (r != LSA_OK) return r;
  }
  return LSA_OK;
}

int lsa_host_stage_bytes(const lsa_params* p, int64_t sq, size_t* bytes) {
  if (bytes == nullptr || sq <= 0) return LSA_ERR_ARG;
  const int r = check_params(p, true, true);
  if (r != LSA_OK) return r;
  if (p->paged || p->n_layers <= 0) return LSA_ERR_ARG;
  size_t off = 0;
  off += align_up(static_cast<size_t>(sq) * p->n_heads_idx * p->d_idx * 2, 256);
  off += align_up(static_cast<size_t>(sq) * p->n_heads_idx * 4, 256);
  off += p->n_layers * align_up(static_cast<size_t>(sq) * p->n_heads * p->d_qk * 2, 256);
  off += p->n_layers * align_up(static_cast<size_t>(sq) * p->n_heads * p->d_v * 2, 256);
  off += align_up(static_cast<size_t>(sq) * p->k_sparse * 4, 256);
  off += align_up(static_cast<size_t>(sq) * 4, 256);
  *bytes = off;
  return LSA_OK;
}

int lsa_layer_group_host(lsa_ctx* c, const lsa_params* p, const void* q_idx_host, const float* w_host,
                         const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query,
                         int64_t n_key, const void* const* q_host, const void* const* k, const void* const* v, int64_t ld_k,
                         int64_t ld_v, void* const* out_host, int64_t sq, void* const* stage, size_t stage_bytes) {
  if (c == nullptr) return LSA_ERR_ARG;
  size_t need = 0;
  int r = lsa_host_stage_bytes(p, sq, &need);
  if (r != LSA_OK) return r;
  if (stage == nullptr || stage[0] == nullptr || stage[1] == nullptr || stage_bytes < need) return LSA_ERR_WORKSPACE;
  if (q_idx_host == nullptr || w_host == nullptr || q_host == nullptr || out_host == nullptr || n_query < 0 || q_pos0 < 0) return LSA_ERR_ARG;
  const int R = p->n_layers;
  if (R > 16) return LSA_ERR_SHAPE;
  const size_t b_qi = static_cast<size_t>(p->n_heads_idx) * p->d_idx * 2, b_w = static_cast<size_t>(p->n_heads_idx) * 4;
  const size_t b_q = static_cast<size_t>(p->n_heads) * p->d_qk * 2, b_o = static_cast<size_t>(p->n_heads) * p->d_v * 2;
  cudaError_t e = cudaSuccess;
  const int64_t n_pass = (n_query + sq - 1) / sq;
  // the caller's earlier work on the context stream must be visible to the copy streams
  e = cudaEventRecord(c->ev_done[0], c->stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(c->copy_in, c->ev_done[0], 0);
  for (int64_t i = 0; i < n_pass && e == cudaSuccess; ++i) {
    const int s = static_cast<int>(i & 1);
    const int64_t q0 = i * sq, n = n_query - q0 < sq ? n_query - q0 : sq;
    uint8_t* base = static_cast<uint8_t*>(stage[s]);
    size_t off = 0;
    uint8_t* d_qi = base + off; off += align_up(static_cast<size_t>(sq) * b_qi, 256);
    uint8_t* d_w = base + off; off += align_up(static_cast<size_t>(sq) * b_w, 256);
    const void* d_q[16]; void* d_o[16];
    for (int l = 0; l < R; ++l) { d_q[l] = base + off; off += align_up(static_cast<size_t>(sq) * b_q, 256); }
    for (int l = 0; l < R; ++l) { d_o[l] = base + off; off += align_up(static_cast<size_t>(sq) * b_o, 256); }
    int32_t* d_idx = reinterpret_cast<int32_t*>(base + off); off += align_up(static_cast<size_t>(sq) * p->k_sparse * 4, 256);
    int32_t* d_n = reinterpret_cast<int32_t*>(base + off);
    // The input half of stage s is free once the kernels of pass i-2 have read it; its output half only once the
    // copy-out of pass i-2 has drained it, which the kernels of this pass (not its copy-in) have to wait for.
    if (i >= 2) e = cudaStreamWaitEvent(c->copy_in, c->ev_done[s], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_qi, static_cast<const uint8_t*>(q_idx_host) + q0 * b_qi, n * b_qi, cudaMemcpyHostToDevice, c->copy_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_w, reinterpret_cast<const uint8_t*>(w_host) + q0 * b_w, n * b_w, cudaMemcpyHostToDevice, c->copy_in);
    for (int l = 0; l < R && e == cudaSuccess; ++l)
      e = cudaMemcpyAsync(const_cast<void*>(d_q[l]), static_cast<const uint8_t*>(q_host[l]) + q0 * b_q, n * b_q, cudaMemcpyHostToDevice, c->copy_in);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_in[s], c->copy_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->stream, c->ev_in[s], 0);
    if (e == cudaSuccess && i >= 2) e = cudaStreamWaitEvent(c->stream, c->ev_out[s], 0);
    if (e != cudaSuccess) break;
    r = lsa_layer_group(c, p, d_qi, reinterpret_cast<const float*>(d_w), k_idx, k_scale, kmean, q_pos0 + q0, n, n_key, nullptr,
                        0, nullptr, 1, d_q, k, v, ld_k, ld_v, d_o, nullptr, d_idx, d_n);
    if (r != LSA_OK) return r;
    e = cudaEventRecord(c->ev_done[s], c->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->copy_out, c->ev_done[s], 0);
    for (int l = 0; l < R && e == cudaSuccess; ++l)
      e = cudaMemcpyAsync(static_cast<uint8_t*>(out_host[l]) + q0 * b_o, d_o[l], n * b_o, cudaMemcpyDeviceToHost, c->copy_out);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_out[s], c->copy_out);
  }
  // the context stream finishes only after every copy-out has
  for (int s = 0; s < 2 && e == cudaSuccess; ++s)
    if (n_pass > s) e = cudaStreamWaitEvent(c->stream, c->ev_out[(n_pass - 1 - s) & 1], 0);
  return e == cudaSuccess ? LSA_OK : cuda_fail(c, e);
}

}  // extern "C"
