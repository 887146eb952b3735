// Host-side launcher interface between the C ABI (lsa_api.cu) and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lsa.h"

namespace lsa {

// Argument checks of an indexer call (parameters, required pointers, ranges, 16-byte alignment of everything the
// kernels read with vector loads); one copy for every entry point that launches the indexer.  Returns an LSA_* code.
int check_index_call(const lsa_params* p, const void* q_idx, const float* w, const void* k_idx, const float* k_scale,
                     const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key, const int32_t* page_table,
                     int64_t page_table_stride, const int32_t* ctx_len, int batch, const int32_t* sparse_idx,
                     const int32_t* n_sparse);

struct IndexArgs {
  int HI, DI, key_e4m3, P, B, M, Ksp, S, W, hi_enable, paged;
  const void* q_idx;      // bf16 [n_query, HI, DI]
  const float* w;         // [n_query, HI]
  const void* k_idx;      // bf16 or e4m3 codes, rows of DI
  const float* k_scale;   // per token, e4m3 only
  const void* k_wide;     // optional: the e4m3 codes widened to bf16 (unscaled), rows of DI, contiguous caches only
  const void* kmean;      // bf16 rows of DI
  int64_t q_pos0;
  int n_query;
  int64_t n_key;
  const int32_t* page_table;
  int64_t pt_stride;
  const int32_t* ctx_len;
  float* page_scores;     // [n_query, ps_ld]
  int ps_ld;
  int32_t* sparse_idx;    // [n_query, Ksp]
  int32_t* n_sparse;
  int32_t* pages_out;     // optional [n_query, M]
  // optional, paged caches: a5 fused into the last selection kernel (what lsa_convert would write)
  int32_t* rows_out;      // [n_query, S + Ksp + W] physical cache rows, -1 padded
  int32_t* n_rows_out;    // [n_query]
  // split fine stage (few queries, many SMs): the scoring blocks leave their results here for the top-K kernel
  int fine_parts;         // 1: fused kernel; >1: blocks per query in the scoring kernel
  uint32_t* fine_keys;    // [n_query, 4096] order-preserving keys of the candidate slots (0 = not a candidate)
  int32_t* fine_pages;    // [n_query, 65]: kept pages, then their count
  int sm_count;           // SMs of the device (grid of the persistent paged kernels)
  int fine_cluster;       // paged caches: the whole fine stage as one clustered tcgen05 kernel (lsa_fine_paged_tc.cu)
  int fine_paged_tc;      // paged caches: page lists, token scores on tcgen05 (lsa_scores_paged_tc.cu), top-K, as three kernels
  int* status;
};

struct AttnArgs {
  int H, DQK, DV, S, W, Ksp, paged;
  float sm_scale;
  const void* q;          // bf16 [n_query, H, DQK]
  const void* k;          // bf16 rows of ld_k
  const void* v;          // bf16 rows of ld_v
  int64_t ld_k, ld_v;
  const int32_t* sparse_idx;
  const int32_t* n_sparse;
  const int32_t* rows;    // optional [n_query, rows_ld]
  const int32_t* n_rows;
  int rows_ld;
  int64_t n_key;          // rows of a contiguous cache (0: paged pool, size unknown); read by the checking build only
  int64_t q_pos0;
  int n_query;
  const int32_t* ctx_len;
  void* out;              // bf16 [n_query, H, DV]
  float* lse;             // optional [n_query, H]
  int pv_issuers;         // tcgen05 kernel: 2 = an issuer owns a lane half (prefill), 4 = one P V issuer per 128 value dims
  int qk_waits_pv;        // tcgen05 kernel, 2 issuers: Q K^T of tile i+1 waits for the completion barrier of P V of tile i-1
  int gather4;            // tcgen05 kernel: scattered rows by TMA gather (cp.async.bulk.tensor tile::gather4) where the cache allows
  int rows_stable;        // tcgen05 kernel, row lists: `rows` / `n_rows` were complete before the previous kernel of the
                          // stream started, so they may be read ahead of the programmatic dependency wait
  int n_split;            // >1: partial results in part_out / part_lse, merged afterwards
  float* part_out;        // fp32 [n_query, n_split, H, DV]
  float* part_lse;        // fp32 [n_query, n_split, H]
  int* status;
};

// Each launcher returns the cudaError_t of its launches and adds the number of kernels it
// launched to *n_launch.
cudaError_t launch_block_means(int DI, int key_e4m3, int B, int kv_page, const void* k_idx, const float* k_scale,
                               int64_t n_key, const int32_t* page_table, int64_t pt_stride,
                               const int32_t* ctx_len, int batch, void* kmean, cudaStream_t st, int64_t* n_launch);
struct AppendArgs {
  int DI, key_e4m3, B, kv_page, batch, n_kv;
  const void* k_new;        // bf16 [batch, DI]
  void* k_idx;
  float* k_scale;
  void* kmean;
  const int32_t* page_table;
  int64_t pt_stride;
  const int32_t* ctx_len;
  int32_t* ctx_len_out;
  const void* kv_new[8];
  void* kv_pool[8];
  int64_t kv_row_bytes;
};
cudaError_t launch_append(const AppendArgs& a, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_coarse(const IndexArgs& a, cudaStream_t st, int64_t* n_launch);
// MinMax pooling (Eq. 13), contiguous caches: extrema cache [ceil(n_key/B), 2*DI] = [k_max | k_min], and the coarse stage on it
cudaError_t launch_block_minmax(int DI, int key_e4m3, int B, const void* k_idx, const float* k_scale, int64_t n_key,
                                void* kminmax, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_coarse_minmax(const IndexArgs& a, cudaStream_t st, int64_t* n_launch);
// tcgen05 version of the coarse stage (contiguous caches, H_I = 64, d_I = 128); groups = 4-query groups per block
bool coarse_tc_supported(const IndexArgs& a);
cudaError_t launch_coarse_tc(const IndexArgs& a, int groups, cudaStream_t st, int64_t* n_launch);
// The coarse stage as every entry point runs it: the tcgen05 kernel where the shape allows, else the mma.sync tile.
inline cudaError_t launch_coarse_best(const IndexArgs& a, int groups, cudaStream_t st, int64_t* n_launch) {
  return coarse_tc_supported(a) ? launch_coarse_tc(a, groups, st, n_launch) : launch_coarse(a, st, n_launch);
}
// tcgen05 version of the coarse stage for paged caches (H_I = 64, d_I = 128); used by launch_coarse
bool fine_paged_tc_supported(const IndexArgs& a);
cudaError_t launch_fine_paged_tc(const IndexArgs& a, int sm_count, cudaStream_t st, int64_t* n_launch);
bool coarse_paged_tc_supported(const IndexArgs& a);
cudaError_t launch_coarse_paged_tc(const IndexArgs& a, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_fine_select(const IndexArgs& a, cudaStream_t st, int64_t* n_launch);
// tcgen05 version of the fine stage's scoring blocks (H_I = 64, d_I = 128); used by launch_fine_select
bool fine_tc_supported(const IndexArgs& a);
cudaError_t launch_fine_select_tc(const IndexArgs& a, cudaStream_t st, int64_t* n_launch);
// Recall budgets M * P > 4096 (contiguous caches, H_I = 64, d_I = 128): page top-M into pages_ws [n_query, M] /
// n_pages_ws [n_query], fine scores as keys [n_query, M * P], top-K_sparse into a.sparse_idx / a.n_sparse
bool fine_big_supported(const IndexArgs& a);
cudaError_t launch_fine_big(const IndexArgs& a, int32_t* pages_ws, int32_t* n_pages_ws, uint32_t* keys, cudaStream_t st,
                            int64_t* n_launch);
// ctx_len != NULL (paged caches): the query of row i sits at ctx_len[i] - 1 instead of q_pos0 + i
cudaError_t launch_select(const float* scores, int64_t ld, const int32_t* cand_pos, const float* pos_scale,
                          int64_t q_pos0, int n_query, int64_t n_cand, int k, int apply_range, int S, int W,
                          int32_t* idx_out, int32_t* n_out, cudaStream_t st, int64_t* n_launch,
                          const int32_t* ctx_len = nullptr);
// Token scores over cache pages on tcgen05 (paged caches, 64-token pages, H_I = 64, d_I = 128).  flat = 0: keys of the
// slots of the page lists a.fine_pages -> a.fine_keys; flat = 1: scores of the whole scoring range -> a.page_scores.
bool paged_scores_tc_supported(const IndexArgs& a);
cudaError_t launch_paged_scores_tc(const IndexArgs& a, int flat, int sm_count, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_widen_e4m3(const void* codes, void* out_bf16, int64_t n_elems, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_convert(int S, int W, int Ksp, int paged, int kv_page, const int32_t* sparse_idx,
                           const int32_t* n_sparse, int64_t q_pos0, int n_query, const int32_t* page_table,
                           int64_t pt_stride, const int32_t* ctx_len, int32_t* rows_out, int32_t* n_rows_out,
                           int32_t* runs_out, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_attn(const AttnArgs& a, cudaStream_t st, int64_t* n_launch);
// tcgen05 version of the attention kernel (MLA latent shape only)
bool attn_tc_supported(const AttnArgs& a);
// row splits that kernel merges itself (clusters of n_split blocks); other counts need launch_merge
bool attn_tc_split_ok(int n_split);
cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t st, int64_t* n_launch);
cudaError_t launch_merge(const AttnArgs& a, cudaStream_t st, int64_t* n_launch);

struct MergeArgs {
  int n_parts, H, DV, n_query;
  const void* outs[8];
  const float* lses[8];
  void* out;
  float* lse;
};
cudaError_t launch_merge_parts(const MergeArgs& a, cudaStream_t st, int64_t* n_launch);

// One block waits on an mbarrier nobody arrives on, for at most budget_cycles (thread 0) before the status word gets
// the time-out code; *waited_ok (optional, zeroed by the caller) counts threads whose wait claimed success.
cudaError_t launch_selftest_wait(int* status, long long budget_cycles, int* waited_ok, cudaStream_t st, int64_t* n_launch);

bool index_shape_supported(int HI, int DI);
bool attn_shape_supported(int H, int DQK, int DV);

}  // namespace lsa
