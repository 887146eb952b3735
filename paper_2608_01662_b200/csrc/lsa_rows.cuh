// Streaming-aware conversion (a5) as device code shared by the kernels that end the indexer: from a query's sparse
// list to the cache rows its attention reads.
#pragma once

#include "lsa_common.cuh"

namespace lsa {

// a5 for one query: cache rows [sink run | sparse ascending | window run] (paged: through the page table), padded
// with -1 to S + Ksp + W entries.  `sparse` may be global memory this block has just written (after a barrier).
// Returns this thread's count of run starts (a row that does not follow its predecessor).
struct RowMap {   // position i of [sink | sparse | window] -> cache row
  int n_sink, n_sp, paged, kv_shift, kv_mask;
  int64_t win0;
  const int32_t* sparse;
  const int32_t* pt;
  __device__ __forceinline__ int32_t operator()(int i) const {
    int64_t pos;
    if (i < n_sink) pos = i;
    else if (i < n_sink + n_sp) pos = sparse[i - n_sink];
    else pos = win0 + (i - n_sink - n_sp);
    return static_cast<int32_t>(paged ? (static_cast<int64_t>(pt[pos >> kv_shift]) << kv_shift) + (pos & kv_mask) : pos);
  }
};

template <int THREADS>
__device__ __forceinline__ int emit_rows(int tid, int S, int W, int Ksp, int paged, int kv_page, const int32_t* sparse,
                                         int n_sp, int64_t t, const int32_t* pt, int32_t* out, bool count_runs) {
  RowMap row_of;
  row_of.n_sink = static_cast<int>(min64(S, t + 1));
  row_of.n_sp = n_sp;
  row_of.paged = paged;
  row_of.kv_shift = paged ? 31 - __clz(kv_page) : 0;   // kv_page is a power of two
  row_of.kv_mask = kv_page - 1;
  row_of.win0 = max64(S, t - W + 1);
  row_of.sparse = sparse;
  row_of.pt = pt;
  const int n_win = static_cast<int>(max64(0, t - row_of.win0 + 1));
  const int n_tot = row_of.n_sink + n_sp + n_win;
  const int ld = S + Ksp + W;
  int breaks = 0;
#pragma unroll 4
  for (int i = tid; i < ld; i += THREADS) {
    int32_t r = -1;
    if (i < n_tot) {
      r = row_of(i);
      if (count_runs && (i == 0 || row_of(i - 1) + 1 != r)) ++breaks;
    }
    out[i] = r;
  }
  return breaks;
}

// Fused a5 at the end of the indexer (paged caches, when the caller asked for it): the rows of query qi from the
// sparse list this block has just written.  In the indexer a cache page is a selection page (kv_page = P).
template <int THREADS>
__device__ __forceinline__ void emit_rows_of_query(int32_t* rows_out, int32_t* n_rows_out, const int32_t* sparse_idx,
                                                   const int32_t* page_table, int64_t pt_stride, int64_t t, int S, int W,
                                                   int Ksp, int paged, int P, int qi, int tid, int n_sel) {
  if (rows_out == nullptr) return;
  const int ld = S + Ksp + W;
  emit_rows<THREADS>(tid, S, W, Ksp, paged, P, sparse_idx + static_cast<int64_t>(qi) * Ksp, n_sel, t,
                     paged ? page_table + qi * pt_stride : nullptr, rows_out + static_cast<int64_t>(qi) * ld, false);
  if (tid == 0) {
    const int n_sink = static_cast<int>(min64(S, t + 1));
    const int64_t win0 = max64(S, t - W + 1);
    n_rows_out[qi] = n_sink + n_sel + static_cast<int>(max64(0, t - win0 + 1));
  }
}

}  // namespace lsa
