// Indexer kernels: sub-block mean cache (a0), coarse page scores (a1, Eq. 9), page top-M (a2, Eq. 10),
// fine token scores on the recalled pages (a3, Eq. 11) and top-K_sparse (a4, Eq. 12), the standalone
// selection (Eq. 2/7) and the streaming-aware conversion of an index set to cache rows (a5, Sec. 3.1).
//
// The scoring kernels of this file are the `mma.sync` forms: they serve the 8-head indexer, paged fine scoring and
// the MinMax variant; the 64-head indexer's coarse and contiguous fine stages run on tcgen05 (lsa_coarse_tc.cu,
// lsa_coarse_paged_tc.cu, lsa_fine_tc.cu, lsa_fine_big_tc.cu).  Also here: the append-token cache maintenance.
//
// Scoring tiles put 128 keys (or mean keys) on the M axis of the tensor-core tile and the H_I heads of
// one query on the N axis, so that the ReLU / head-weight / head-sum epilogue of Eq. 1 runs inside one
// thread quad and one number per key leaves the tile.
#include "lsa_internal.h"
#include "lsa_select.cuh"
#include "lsa_select_cluster.cuh"
#include "lsa_rows.cuh"

#ifdef LSA_TIMELINE
// Debug build only: SM-clock stamps of the fine kernel's phases per block, read back with lsa_debug_timeline_fine.
__device__ long long g_tl_fine[1024 * 8];
#define LSA_TLF(k)                                                              \
  do {                                                                          \
    const unsigned blk_ = blockIdx.x + gridDim.x * blockIdx.y;                  \
    if (threadIdx.x == 0 && blk_ < 1024) g_tl_fine[blk_ * 8 + (k)] = clock64(); \
  } while (0)
extern "C" __attribute__((visibility("default"))) int lsa_debug_timeline_fine(long long* host, int n_blocks) {
  return cudaMemcpyFromSymbol(host, g_tl_fine, sizeof(long long) * 8 * (n_blocks < 1024 ? n_blocks : 1024)) == cudaSuccess ? 0 : -1;
}
#else
#define LSA_TLF(k)
#endif

namespace lsa {

namespace {

constexpr int kTileRows = 128;   // keys per scoring tile
constexpr int kThreads = 256;    // 8 warps, 16 tile rows each

// ------------------------------------------------------------------------------------------------
// a0: mean-key cache
// ------------------------------------------------------------------------------------------------
template <bool E4M3>
__global__ void block_means_kernel(const uint8_t* __restrict__ k_idx, const float* __restrict__ k_scale,
                                   int64_t n_key, int DI, int B, int kv_page,
                                   const int32_t* __restrict__ page_table, int64_t pt_stride,
                                   const int32_t* __restrict__ ctx_len, __nv_bfloat16* __restrict__ kmean) {
  const int U = DI / 8;  // 8 output dims per thread
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t sub = gid / U;
  const int u = static_cast<int>(gid % U);
  int64_t row0, out_row;
  int cnt;
  if (page_table != nullptr) {
    const int b = blockIdx.y;
    const int64_t n = ctx_len[b];
    if (sub * B >= n) return;
    const int64_t pos0 = sub * B;
    const int64_t phys = page_table[b * pt_stride + pos0 / kv_page];
    row0 = phys * kv_page + pos0 % kv_page;
    out_row = phys * (kv_page / B) + (pos0 % kv_page) / B;
    cnt = static_cast<int>(min64(B, n - pos0));
  } else {
    if (sub * B >= n_key) return;
    row0 = sub * B;
    out_row = sub;
    cnt = static_cast<int>(min64(B, n_key - row0));
  }
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int r = 0; r < cnt; ++r) {
    const int64_t row = row0 + r;
    if (E4M3) {
      const uint2 c = *reinterpret_cast<const uint2*>(k_idx + row * DI + u * 8);
      const float sc = k_scale[row];
      const uint32_t w[2] = {c.x, c.y};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(
            static_cast<__nv_fp8x2_storage_t>((w[j >> 1] >> ((j & 1) * 16)) & 0xffff), __NV_E4M3);
        const float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
        acc[2 * j] += f.x * sc;
        acc[2 * j + 1] += f.y * sc;
      }
    } else {
      const uint4 c = *reinterpret_cast<const uint4*>(k_idx + (row * DI + u * 8) * 2);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(h[j]);
        acc[2 * j] += f.x;
        acc[2 * j + 1] += f.y;
      }
    }
  }
  const float inv = static_cast<float>(cnt);
  uint4 o;
  o.x = pack_bf16(acc[0] / inv, acc[1] / inv);
  o.y = pack_bf16(acc[2] / inv, acc[3] / inv);
  o.z = pack_bf16(acc[4] / inv, acc[5] / inv);
  o.w = pack_bf16(acc[6] / inv, acc[7] / inv);
  *reinterpret_cast<uint4*>(kmean + out_row * DI + u * 8) = o;
}

// ------------------------------------------------------------------------------------------------
// shared scoring pieces
// ------------------------------------------------------------------------------------------------

// Copy one query's indexer heads [HI, DI] bf16 (contiguous) into a swizzled shared tile.
template <int HI, int DI>
__device__ __forceinline__ void load_q_async(uint32_t dst, const __nv_bfloat16* src) {
  constexpr int U = DI / 8;
  for (int e = threadIdx.x; e < HI * U; e += kThreads)
    cp_async16(dst + swz<DI * 2>(e / U, e % U), reinterpret_cast<const uint8_t*>(src) + e * 16, 16);
}

// A fragments of this warp's 16 rows of a [128, DI] swizzled tile.
template <int DI>
__device__ __forceinline__ void load_a_frags(uint32_t (&a)[DI / 16][4], uint32_t tile) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = 16 * warp + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
  for (int ks = 0; ks < DI / 16; ++ks) ldmatrix_x4(a[ks], tile + swz<DI * 2>(row, 2 * ks + (lane >> 4)));
}

// Eq. 1 for the warp's rows g and g+8:  sum_j w[j] * relu(row . q_j).  Every lane of a quad gets
// the finished sums.
template <int HI, int DI>
__device__ __forceinline__ void score_16rows(const uint32_t (&a)[DI / 16][4], uint32_t q_tile,
                                             const float* __restrict__ ws, float& s_lo, float& s_hi) {
  constexpr int NT = HI / 8, KS = DI / 16;
  const int lane = threadIdx.x & 31;
  float acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    if constexpr (NT == 1) {
      uint32_t b[2];
      ldmatrix_x2(b, q_tile + swz<DI * 2>(lane & 7, 2 * ks + ((lane >> 3) & 1)));
      mma_bf16(acc[0], a[ks], b[0], b[1]);
    } else {
#pragma unroll
      for (int nt = 0; nt < NT; nt += 2) {
        uint32_t b[4];
        ldmatrix_x4(b, q_tile + swz<DI * 2>(8 * nt + (lane & 7) + (lane >> 4) * 8, 2 * ks + ((lane >> 3) & 1)));
        mma_bf16(acc[nt], a[ks], b[0], b[1]);
        mma_bf16(acc[nt + 1], a[ks], b[2], b[3]);
      }
    }
  }
  const int c2 = (lane & 3) * 2;
  s_lo = 0.f;
  s_hi = 0.f;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const float w0 = ws[8 * nt + c2], w1 = ws[8 * nt + c2 + 1];
    s_lo = fmaf(w0, fmaxf(acc[nt][0], 0.f), s_lo);
    s_lo = fmaf(w1, fmaxf(acc[nt][1], 0.f), s_lo);
    s_hi = fmaf(w0, fmaxf(acc[nt][2], 0.f), s_hi);
    s_hi = fmaf(w1, fmaxf(acc[nt][3], 0.f), s_hi);
  }
  s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1);
  s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1);
  s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
  s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);
}

// ------------------------------------------------------------------------------------------------
// a1: coarse page scores (Eq. 9).  One block = one tile of 128 mean keys x a group of queries.
// ------------------------------------------------------------------------------------------------
constexpr int kCoarseQG = 32;  // prefill queries per block

template <int HI, int DI>
struct CoarseSmem {
  alignas(128) uint8_t a[kTileRows * DI * 2];
  alignas(128) uint8_t q[2][HI * DI * 2];
  float w[2][HI];
  float sub[kTileRows];
};

template <int HI, int DI>
__global__ void __launch_bounds__(kThreads) coarse_score_kernel(IndexArgs p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  auto& sm = *reinterpret_cast<CoarseSmem<HI, DI>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int spp = p.P / p.B;          // sub-blocks per page
  const int ppt = kTileRows / spp;    // pages per tile
  const int64_t sub0 = static_cast<int64_t>(blockIdx.x) * kTileRows;
  const int64_t page0 = sub0 / spp;

  int q_begin, q_end;
  int64_t n_key;
  const int32_t* pt = nullptr;
  if (p.paged) {
    q_begin = blockIdx.y;
    q_end = q_begin + 1;
    n_key = p.ctx_len[q_begin];
    pt = p.page_table + q_begin * p.pt_stride;
  } else {
    q_begin = blockIdx.y * kCoarseQG;
    q_end = min(p.n_query, q_begin + kCoarseQG);
    n_key = p.n_key;
  }
  auto pos_of = [&](int qi) -> int64_t { return p.paged ? n_key - 1 : p.q_pos0 + qi; };
  // A query needs this tile iff the tile's first page is eligible (page0*P <= t-W) and the coarse
  // stage runs at all for it (more than M eligible pages).
  const int64_t t_need = max(page0 * p.P + p.W, (static_cast<int64_t>(p.M) + p.S / p.P) * p.P + p.W);
  if (pos_of(q_end - 1) < t_need) return;
  int q_first = q_begin;
  if (!p.paged && t_need - p.q_pos0 > q_begin) q_first = static_cast<int>(t_need - p.q_pos0);

  // ---- mean-key tile -> shared (zero rows past the end of the cache)
  const int64_t n_sub = (n_key + p.B - 1) / p.B;
  {
    constexpr int U = DI / 8;
    const uint8_t* km = reinterpret_cast<const uint8_t*>(p.kmean);
    for (int e = tid; e < kTileRows * U; e += kThreads) {
      const int r = e / U, u = e % U;
      const int64_t sub = sub0 + r;
      int64_t src_row = sub;
      if (p.paged && sub < n_sub) src_row = static_cast<int64_t>(pt[sub / spp]) * spp + sub % spp;
      cp_async16(smem_u32(sm.a) + swz<DI * 2>(r, u), km + (sub < n_sub ? src_row : 0) * DI * 2 + u * 16,
                 sub < n_sub ? 16 : 0);
    }
  }
  const __nv_bfloat16* qg = reinterpret_cast<const __nv_bfloat16*>(p.q_idx);
  auto prefetch_q = [&](int qi, int buf) {
    load_q_async<HI, DI>(smem_u32(sm.q[buf]), qg + static_cast<int64_t>(qi) * HI * DI);
    if (tid < HI / 4) cp_async16(smem_u32(&sm.w[buf][tid * 4]), p.w + static_cast<int64_t>(qi) * HI + tid * 4, 16);
    cp_async_commit();
  };
  prefetch_q(q_first, 0);
  cp_async_wait<0>();
  __syncthreads();
  uint32_t a[DI / 16][4];
  load_a_frags<DI>(a, smem_u32(sm.a));

  for (int qi = q_first; qi < q_end; ++qi) {
    const int buf = (qi - q_first) & 1;
    if (qi + 1 < q_end) prefetch_q(qi + 1, buf ^ 1);
    float s_lo, s_hi;
    score_16rows<HI, DI>(a, smem_u32(sm.q[buf]), sm.w[buf], s_lo, s_hi);
    if ((lane & 3) == 0) {
      sm.sub[16 * warp + (lane >> 2)] = s_lo;
      sm.sub[16 * warp + (lane >> 2) + 8] = s_hi;
    }
    __syncthreads();
    if (tid < ppt) {
      const int64_t page = page0 + tid;
      const int64_t hi = pos_of(qi) - p.W;
      if (page * p.P <= hi) {
        float s = 0.f;
        for (int j = 0; j < spp; ++j) s += sm.sub[tid * spp + j];
        p.page_scores[static_cast<int64_t>(qi) * p.ps_ld + page] = s;
      }
    }
    cp_async_wait<0>();
    __syncthreads();
  }
}

// Paged (decode) form of a1: one query per sequence, so a block keeps the query resident and streams several
// mean-key tiles of that sequence through a three-deep ring (the mean cache is the large operand here: the stage
// is an HBM read of the whole cache of means, and a tile costs a page-table look-up plus an HBM round trip, so two
// blocks per SM with two tiles each in flight are what keeps the memory pipe full).
constexpr int kCoarseTilesPerBlock = 8;
constexpr int kCoarseStages = 3;

template <int HI, int DI>
struct CoarsePagedSmem {
  alignas(128) uint8_t a[kCoarseStages][kTileRows * DI * 2];
  alignas(128) uint8_t q[HI * DI * 2];
  float w[HI];
  float sub[kTileRows];
};

template <int HI, int DI>
__global__ void __launch_bounds__(kThreads, 2) coarse_score_paged_kernel(IndexArgs p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  auto& sm = *reinterpret_cast<CoarsePagedSmem<HI, DI>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.y;
  const int64_t n_key = p.ctx_len[qi];
  const int64_t t = n_key - 1, hi = t - p.W;
  const int spp = p.P / p.B, ppt = kTileRows / spp;
  // the coarse stage runs only when more than M pages are eligible
  if (hi < p.S || hi / p.P - p.S / p.P + 1 <= p.M) return;
  const int64_t n_sub = (n_key + p.B - 1) / p.B;
  const int tiles_needed = static_cast<int>(hi / p.P / ppt) + 1;   // tiles holding an eligible page
  const int tile_begin = blockIdx.x * kCoarseTilesPerBlock;
  const int tile_end = min(tiles_needed, tile_begin + kCoarseTilesPerBlock);
  if (tile_begin >= tile_end) return;
  const int32_t* pt = p.page_table + qi * p.pt_stride;
  const uint8_t* km = reinterpret_cast<const uint8_t*>(p.kmean);
  const int spp_shift = 31 - __clz(spp);   // spp is 8, 16 or 32
  constexpr int U = DI / 8;
  constexpr int kPer = kTileRows * U / kThreads;   // 16-byte chunks per thread and tile
  auto issue_tile = [&](int tile, int buf) {
    // page-table look-ups first, all in flight together; then the copies that depend on them
    int64_t src_row[kPer];
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
      const int r = (tid + j * kThreads) / U;
      const int sub = tile * kTileRows + r;   // sub-block number (fits 32 bits: cache lengths do)
      src_row[j] = sub < n_sub ? (static_cast<int64_t>(pt[sub >> spp_shift]) << spp_shift) + (sub & (spp - 1)) : -1;
    }
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
      const int e = tid + j * kThreads, r = e / U, u = e % U;
      const bool ok = src_row[j] >= 0;
      cp_async16(smem_u32(sm.a[buf]) + swz<DI * 2>(r, u), km + (ok ? src_row[j] : 0) * DI * 2 + u * 16, ok ? 16 : 0);
    }
    cp_async_commit();
  };
  load_q_async<HI, DI>(smem_u32(sm.q), reinterpret_cast<const __nv_bfloat16*>(p.q_idx) + static_cast<int64_t>(qi) * HI * DI);
  if (tid < HI / 4) cp_async16(smem_u32(&sm.w[tid * 4]), p.w + static_cast<int64_t>(qi) * HI + tid * 4, 16);
  // one cp.async group per tile, also when there is no tile left (an empty group), so the wait depth is constant
  for (int j = 0; j < kCoarseStages - 1; ++j) {
    if (tile_begin + j < tile_end) issue_tile(tile_begin + j, j);
    else cp_async_commit();
  }
  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int buf = (tile - tile_begin) % kCoarseStages;
    // the buffer refilled here was read two iterations ago; the barrier that ended that iteration covers it
    if (tile + kCoarseStages - 1 < tile_end) issue_tile(tile + kCoarseStages - 1, (buf + kCoarseStages - 1) % kCoarseStages);
    else cp_async_commit();
    cp_async_wait<kCoarseStages - 1>();
    __syncthreads();   // tile (and, first time, q / w) in shared
    uint32_t a[DI / 16][4];
    load_a_frags<DI>(a, smem_u32(sm.a[buf]));
    float s_lo, s_hi;
    score_16rows<HI, DI>(a, smem_u32(sm.q), sm.w, s_lo, s_hi);
    if ((lane & 3) == 0) {
      sm.sub[16 * warp + (lane >> 2)] = s_lo;
      sm.sub[16 * warp + (lane >> 2) + 8] = s_hi;
    }
    __syncthreads();
    if (tid < ppt) {
      const int64_t page = static_cast<int64_t>(tile) * ppt + tid;
      if (page * p.P <= hi) {
        float s = 0.f;
        for (int j = 0; j < spp; ++j) s += sm.sub[tid * spp + j];
        p.page_scores[static_cast<int64_t>(qi) * p.ps_ld + page] = s;
      }
    }
    __syncthreads();   // sub and buffer `buf` are reused two tiles on
  }
}

// ------------------------------------------------------------------------------------------------
// a2-a4: per query: top-M pages, fine scores on their tokens, top-K_sparse.
// ------------------------------------------------------------------------------------------------
constexpr int kClusterRowsMax = 256;    // rows: up to this many, a row of kClusterMinRow scores or more gets a cluster of blocks
constexpr int kClusterMinRow = 16384;
constexpr int kMaxSlots = 4096;  // keep_pages * page
constexpr int kMaxPages = 64;    // keep_pages

template <int HI, int DI>
struct FineSmem {
  alignas(128) uint8_t a[2][kTileRows * DI * 2];
  alignas(128) uint8_t q[HI * DI * 2];
  float w[HI];
  uint32_t keys[kMaxSlots];
  float scale[2][kTileRows];   // per-token key scales of the tile in flight (e4m3 keys)
  int32_t pages[kMaxPages];
  int32_t phys[kMaxPages];     // where each selected page lives in the cache (page-table entry; the page itself when contiguous)
  SelectScratch sel;
};

template <int HI, int DI, bool E4M3>
__global__ void __launch_bounds__(kThreads, 2) fine_select_kernel(IndexArgs p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  auto& sm = *reinterpret_cast<FineSmem<HI, DI>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.x;
  LSA_TLF(0);
  pdl_wait();
  pdl_launch_dependents();
  LSA_TLF(1);
  int64_t t, n_key;
  const int32_t* pt = nullptr;
  if (p.paged) {
    n_key = p.ctx_len[qi];
    t = n_key - 1;
    pt = p.page_table + qi * p.pt_stride;
  } else {
    n_key = p.n_key;
    t = p.q_pos0 + qi;
  }
  int32_t* out_idx = p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp;
  int32_t* out_pages = p.pages_out ? p.pages_out + static_cast<int64_t>(qi) * p.M : nullptr;
  const int64_t lo = p.S, hi = t - p.W;
  const int part = blockIdx.y, n_parts = gridDim.y;   // > 1: this block scores a share of the tiles only
  if (hi < lo) {
    if (part != 0) return;
    if (n_parts > 1) p.fine_pages[qi * (kMaxPages + 1) + kMaxPages] = 0;
    for (int i = tid; i < p.Ksp; i += kThreads) out_idx[i] = -1;
    if (out_pages) for (int i = tid; i < p.M; i += kThreads) out_pages[i] = -1;
    if (tid == 0) p.n_sparse[qi] = 0;
    emit_rows_of_query<kThreads>(p.rows_out, p.n_rows_out, p.sparse_idx, p.page_table, p.pt_stride, t, p.S, p.W, p.Ksp, p.paged,
                                 p.P, qi, tid, 0);
    return;
  }
  const int p0 = static_cast<int>(lo / p.P), p1 = static_cast<int>(hi / p.P);
  const int nE = p1 - p0 + 1;
  int nP;
  if (p.hi_enable && nE > p.M) {
    const float* ps = p.page_scores + static_cast<int64_t>(qi) * p.ps_ld + p0;
    if (nE <= kMaxSlots) {
      // one pass over the page scores (L2) into the candidate buffer, which is idle until the fine stage;
      // the six passes of the radix select then run out of shared memory
      for (int i = tid; i < nE; i += kThreads) sm.keys[i] = score_key(ps[i]);
      __syncthreads();
      LSA_TLF(7);
      nP = block_select_topk([&](int i) { return sm.keys[i]; }, [&](int i) { return p0 + i; }, nE, p.M, sm.pages, sm.sel);
    } else {
      nP = block_select_topk<0, true>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M,
                             sm.pages, sm.sel);
    }
  } else {
    nP = nE;  // host guarantees nE <= kMaxSlots / P here
    for (int i = tid; i < nP; i += kThreads) sm.pages[i] = p0 + i;
  }
  LSA_TLF(2);
  // ---- query heads and weights -> shared
  load_q_async<HI, DI>(smem_u32(sm.q), reinterpret_cast<const __nv_bfloat16*>(p.q_idx) + static_cast<int64_t>(qi) * HI * DI);
  if (tid < HI / 4) cp_async16(smem_u32(&sm.w[tid * 4]), p.w + static_cast<int64_t>(qi) * HI + tid * 4, 16);
  cp_async_commit();
  __syncthreads();  // sm.pages visible
  // one page-table lookup per selected page, not one per copied chunk
  for (int i = tid; i < nP; i += kThreads) sm.phys[i] = p.paged ? pt[sm.pages[i]] : sm.pages[i];
  __syncthreads();
  if (out_pages && part == 0) for (int i = tid; i < p.M; i += kThreads) out_pages[i] = i < nP ? sm.pages[i] : -1;
  if (n_parts > 1 && part == 0) {
    int32_t* fp = p.fine_pages + qi * (kMaxPages + 1);
    for (int i = tid; i < nP; i += kThreads) fp[i] = sm.pages[i];
    if (tid == 0) fp[kMaxPages] = nP;
  }

  const int n_slots = nP * p.P;
  const int n_tiles_all = (n_slots + kTileRows - 1) / kTileRows;
  const int tiles_per = (n_tiles_all + n_parts - 1) / n_parts;
  const int tile0 = part * tiles_per;
  const int n_tiles = max(0, min(n_tiles_all, tile0 + tiles_per) - tile0);
  const int pshift = 31 - __clz(p.P);
  auto slot_pos = [&](int c) -> int64_t { return static_cast<int64_t>(sm.pages[c >> pshift]) * p.P + (c & (p.P - 1)); };
  auto slot_row = [&](int c) -> int64_t { return static_cast<int64_t>(sm.phys[c >> pshift]) * p.P + (c & (p.P - 1)); };
  const uint8_t* kbase = reinterpret_cast<const uint8_t*>(p.k_idx);

  // Tile loaders.  bf16 keys go global -> shared asynchronously; e4m3 keys are read into registers one
  // tile ahead, widened to bf16 and stored.
  constexpr int U = DI / 8;                           // 16-byte bf16 units per row
  constexpr int CU = DI / 16;                         // 16-byte code units per row (e4m3)
  constexpr int kCodePerThread = kTileRows * CU / kThreads;
  // e4m3: kDepth tiles are in flight in registers (a gathered tile takes several microseconds to arrive from a
  // multi-GB cache; one tile ahead left the loop waiting on it)
  constexpr int kDepth = E4M3 ? 3 : 1;
  uint4 staged_all[kDepth][E4M3 ? kCodePerThread : 1];
  float staged_scale_all[kDepth];
  auto issue_tile = [&](int tile, int buf, uint4* staged, float& staged_scale) {
    if constexpr (E4M3) {
      if (tid < kTileRows) {   // this row's scale travels with the tile instead of being fetched after the MMAs
        const int c = tile * kTileRows + tid;
        staged_scale = 0.f;
        if (c < n_slots) {
          const int64_t pos = slot_pos(c);
          if (pos < n_key) staged_scale = p.k_scale[slot_row(c)];
        }
      }
#pragma unroll
      for (int j = 0; j < kCodePerThread; ++j) {
        const int e = tid + j * kThreads, r = e / CU, u = e % CU;
        const int c = tile * kTileRows + r;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (c < n_slots) {
          const int64_t pos = slot_pos(c);
          if (pos < n_key) v = *reinterpret_cast<const uint4*>(kbase + slot_row(c) * DI + u * 16);
        }
        staged[j] = v;
      }
    } else {
      for (int e = tid; e < kTileRows * U; e += kThreads) {
        const int r = e / U, u = e % U;
        const int c = tile * kTileRows + r;
        bool ok = c < n_slots;
        int64_t pos = 0;
        if (ok) {
          pos = slot_pos(c);
          ok = pos < n_key;
        }
        cp_async16(smem_u32(sm.a[buf]) + swz<DI * 2>(r, u), kbase + (ok ? slot_row(c) : 0) * DI * 2 + u * 16,
                   ok ? 16 : 0);
      }
      cp_async_commit();
    }
  };
  auto land_tile = [&](int buf, const uint4* staged, float staged_scale) {
    if constexpr (E4M3) {
      if (tid < kTileRows) sm.scale[buf][tid] = staged_scale;
#pragma unroll
      for (int j = 0; j < kCodePerThread; ++j) {
        const int e = tid + j * kThreads, r = e / CU, u = e % CU;
        uint4 lo16, hi16;
        e4m3x16_to_bf16(staged[j], lo16, hi16);
        *reinterpret_cast<uint4*>(sm.a[buf] + swz<DI * 2>(r, 2 * u)) = lo16;
        *reinterpret_cast<uint4*>(sm.a[buf] + swz<DI * 2>(r, 2 * u + 1)) = hi16;
      }
    }
  };

#pragma unroll
  for (int d = 0; d < kDepth; ++d)
    if (d < n_tiles) issue_tile(tile0 + d, d & 1, staged_all[d], staged_scale_all[d]);
  for (int base = 0; base < n_tiles; base += kDepth) {
#pragma unroll
   for (int d = 0; d < kDepth; ++d) {
    const int it = base + d;           // block-uniform
    if (it >= n_tiles) break;
    const int tile = tile0 + it;
    const int buf = it & 1;
    land_tile(buf, staged_all[d], staged_scale_all[d]);
    cp_async_wait<0>();
    __syncthreads();  // tile `tile` (and, first time, q/w) in shared; buffer buf^1 free
    if (it == 0) LSA_TLF(3);
    if (it == 3) LSA_TLF(4);
    if (it + kDepth < n_tiles) issue_tile(tile + kDepth, (it + kDepth) & 1, staged_all[d], staged_scale_all[d]);
    uint32_t a[DI / 16][4];
    load_a_frags<DI>(a, smem_u32(sm.a[buf]));
    float s_lo, s_hi;
    score_16rows<HI, DI>(a, smem_u32(sm.q), sm.w, s_lo, s_hi);
    if ((lane & 3) == 0) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int c = tile * kTileRows + 16 * warp + (lane >> 2) + 8 * half;
        if (c < n_slots) {
          const int64_t pos = slot_pos(c);
          uint32_t key = 0;
          if (pos >= lo && pos <= hi) {
            float s = half ? s_hi : s_lo;
            if constexpr (E4M3) s *= sm.scale[buf][16 * warp + (lane >> 2) + 8 * half];
            key = score_key(s);
          }
          sm.keys[c] = key;
        }
      }
    }
   }
  }
  __syncthreads();
  LSA_TLF(5);
  if (n_parts > 1) {
    // hand this block's share of the candidate keys to the top-K kernel
    uint32_t* fk = p.fine_keys + static_cast<int64_t>(qi) * kMaxSlots;
    const int c0 = tile0 * kTileRows, c1 = min(n_slots, (tile0 + n_tiles) * kTileRows);
    for (int c = c0 + tid; c < c1; c += kThreads) fk[c] = sm.keys[c];
    LSA_TLF(6);
    return;
  }
  const int n_sel = block_select_topk([&](int i) { return sm.keys[i]; },
                                      [&](int i) { return static_cast<int>(slot_pos(i)); }, n_slots, p.Ksp, out_idx,
                                      sm.sel);
  if (tid == 0) p.n_sparse[qi] = n_sel;
  // (rows_out: the caller runs convert_kernel after an unsplit launch; a call to the row writer at this point of the
  // template trips an internal error of nvcc 12.9)
}

// a2 for paged caches as a kernel of its own (the tcgen05 scoring kernel that follows walks ready-made page lists):
// the pages of sequence qi that survive the coarse stage (Eq. 10), ascending, into fine_pages[qi], their count last.
// A sequence without candidates gets its (empty) results here.
__global__ void __launch_bounds__(kSelThreads) page_topm_paged_kernel(IndexArgs p) {
  __shared__ uint32_t keys[kMaxSlots];
  __shared__ int32_t pages[kMaxPages];
  __shared__ SelectScratch sc;
  const int qi = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const int64_t t = static_cast<int64_t>(p.ctx_len[qi]) - 1;
  const int64_t lo = p.S, hi = t - p.W;
  int32_t* fp = p.fine_pages + qi * (kMaxPages + 1);
  int32_t* out_pages = p.pages_out ? p.pages_out + static_cast<int64_t>(qi) * p.M : nullptr;
  if (hi < lo) {
    if (tid == 0) {
      fp[kMaxPages] = 0;
      p.n_sparse[qi] = 0;
    }
    for (int i = tid; i < p.Ksp; i += kSelThreads) p.sparse_idx[static_cast<int64_t>(qi) * p.Ksp + i] = -1;
    if (out_pages) for (int i = tid; i < p.M; i += kSelThreads) out_pages[i] = -1;
    emit_rows_of_query<kSelThreads>(p.rows_out, p.n_rows_out, p.sparse_idx, p.page_table, p.pt_stride, t, p.S, p.W, p.Ksp, p.paged,
                                    p.P, qi, tid, 0);
    return;
  }
  const int p0 = static_cast<int>(lo / p.P), p1 = static_cast<int>(hi / p.P);
  const int nE = p1 - p0 + 1;
  int nP;
  if (p.hi_enable && nE > p.M) {
    const float* ps = p.page_scores + static_cast<int64_t>(qi) * p.ps_ld + p0;
    if (nE <= kMaxSlots) {
      for (int i = tid; i < nE; i += kSelThreads) keys[i] = score_key(ps[i]);
      __syncthreads();
      nP = block_select_topk([&](int i) { return keys[i]; }, [&](int i) { return p0 + i; }, nE, p.M, pages, sc);
    } else {
      nP = block_select_topk<0, true>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M, pages, sc);
    }
  } else {
    nP = nE;   // the host guarantees nE <= kMaxPages here
    for (int i = tid; i < nP; i += kSelThreads) pages[i] = p0 + i;
    __syncthreads();
  }
  for (int i = tid; i < nP; i += kSelThreads) fp[i] = pages[i];
  if (tid == 0) fp[kMaxPages] = nP;
  if (out_pages) for (int i = tid; i < p.M; i += kSelThreads) out_pages[i] = i < nP ? pages[i] : -1;
}

// Second half of the split fine stage: top-K_sparse over the keys the scoring blocks left in global memory.
__global__ void __launch_bounds__(kSelThreads) fine_topk_kernel(IndexArgs p) {
  __shared__ uint32_t keys[kMaxSlots];
  __shared__ int32_t pages[kMaxPages];
  __shared__ SelectScratch sc;
  const int qi = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const int32_t* fp = p.fine_pages + qi * (kMaxPages + 1);
  const int nP = fp[kMaxPages];
  if (nP == 0) return;   // no candidates: the scoring kernel has written the empty result
  const int n_slots = nP * p.P;
  const uint32_t* fk = p.fine_keys + static_cast<int64_t>(qi) * kMaxSlots;
  for (int i = tid; i < n_slots; i += kSelThreads) keys[i] = fk[i];
  for (int i = tid; i < nP; i += kSelThreads) pages[i] = fp[i];
  __syncthreads();
  const int pshift = 31 - __clz(p.P);
  const int n_sel = block_select_topk([&](int i) { return keys[i]; },
                                      [&](int i) { return pages[i >> pshift] * p.P + (i & (p.P - 1)); }, n_slots, p.Ksp,
                                      p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp, sc);
  if (tid == 0) p.n_sparse[qi] = n_sel;
  // the select ended with a barrier: the list is visible to the block
  emit_rows_of_query<kSelThreads>(p.rows_out, p.n_rows_out, p.sparse_idx, p.page_table, p.pt_stride,
                                  p.paged ? static_cast<int64_t>(p.ctx_len[qi]) - 1 : p.q_pos0 + qi, p.S, p.W, p.Ksp, p.paged,
                                  p.P, qi, tid, n_sel);
}

// ------------------------------------------------------------------------------------------------
// standalone selection on caller-given scores
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads) select_kernel(const float* __restrict__ scores, int64_t ld,
                                                            const int32_t* __restrict__ cand_pos,
                                                            const float* __restrict__ pos_scale, int64_t q_pos0,
                                                            int64_t n_cand, int k, int apply_range, int S, int W,
                                                            int32_t* __restrict__ idx_out, int32_t* __restrict__ n_out,
                                                            const int32_t* __restrict__ ctx_len) {
  __shared__ SelectScratch sc;
  const int qi = blockIdx.x;
  const float* row = scores + qi * ld;
  const int32_t* pos = cand_pos ? cand_pos + qi * n_cand : nullptr;
  // the query of row qi sits at q_pos0 + qi, or (paged caches: one query per sequence) at the end of its sequence
  const int64_t lo = S, hi = (ctx_len ? static_cast<int64_t>(ctx_len[qi]) - 1 : q_pos0 + qi) - W;
  auto id = [&](int i) { return pos ? pos[i] : i; };
  // (no branch between the loads and the test: the caller evaluates several keys per step and wants their loads in
  // flight together)
  auto key = [&](int i) -> uint32_t {
    const int64_t s = id(i);
    const bool ok = s >= 0 && (!apply_range || (s >= lo && s <= hi));
    float v = row[i];
    // pos_scale: per-position factor of the score (the fp32 scale of an e4m3 key), applied before the comparison
    if (pos_scale) v *= pos_scale[s < 0 ? 0 : s];
    return ok ? score_key(v) : 0u;
  };
  // columns that are positions: nothing beyond the range can take part, so it is not even scanned
  int n = static_cast<int>(n_cand);
  if (pos == nullptr && apply_range) n = static_cast<int>(max64(0, min64(n_cand, hi + 1)));
  const int n_sel = block_select_topk<0, true>(key, id, n, k, idx_out + static_cast<int64_t>(qi) * k, sc);
  if (threadIdx.x == 0) n_out[qi] = n_sel;
}

// The same selection with a cluster of kClusterSel blocks per row (few long rows: the flat indexer in decode).
__global__ void __launch_bounds__(kSelThreads) select_cluster_kernel(const float* __restrict__ scores, int64_t ld,
                                                                    const int32_t* __restrict__ cand_pos,
                                                                    const float* __restrict__ pos_scale, int64_t q_pos0,
                                                                    int64_t n_cand, int k, int apply_range, int S, int W,
                                                                    int32_t* __restrict__ idx_out, int32_t* __restrict__ n_out,
                                                                    const int32_t* __restrict__ ctx_len) {
  __shared__ ClusterSelScratch sc;
  const int qi = blockIdx.y;
  const float* row = scores + qi * ld;
  const int32_t* pos = cand_pos ? cand_pos + qi * n_cand : nullptr;
  const int64_t lo = S, hi = (ctx_len ? static_cast<int64_t>(ctx_len[qi]) - 1 : q_pos0 + qi) - W;
  auto id = [&](int i) { return pos ? pos[i] : i; };
  auto key = [&](int i) -> uint32_t {   // branch-free, as in select_kernel
    const int64_t s = id(i);
    const bool ok = s >= 0 && (!apply_range || (s >= lo && s <= hi));
    float v = row[i];
    if (pos_scale) v *= pos_scale[s < 0 ? 0 : s];
    return ok ? score_key(v) : 0u;
  };
  int n = static_cast<int>(n_cand);
  if (pos == nullptr && apply_range) n = static_cast<int>(max64(0, min64(n_cand, hi + 1)));
  const int n_sel = cluster_select_topk(key, id, n, k, idx_out + static_cast<int64_t>(qi) * k, sc);
  if (threadIdx.x == 0 && blockIdx.x == 0) n_out[qi] = n_sel;
}

// e4m3 codes -> the same values as bf16 (exact), for the dense scoring of the flat indexer
__global__ void widen_e4m3_kernel(const uint4* __restrict__ codes, uint4* __restrict__ out, int64_t n_units) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n_units) return;
  uint4 lo16, hi16;
  e4m3x16_to_bf16(codes[i], lo16, hi16);
  out[2 * i] = lo16;
  out[2 * i + 1] = hi16;
}

// ------------------------------------------------------------------------------------------------
// a5: index set -> cache rows  [sink run | sparse ascending | window run]
// ------------------------------------------------------------------------------------------------
constexpr int kConvertThreads = 1024;   // every row of a query has its own thread or nearly: the look-ups are two dependent loads

__global__ void __launch_bounds__(kConvertThreads) convert_kernel(int S, int W, int Ksp, int paged, int kv_page,
                                                     const int32_t* __restrict__ sparse_idx,
                                                     const int32_t* __restrict__ n_sparse, int64_t q_pos0,
                                                     const int32_t* __restrict__ page_table, int64_t pt_stride,
                                                     const int32_t* __restrict__ ctx_len,
                                                     int32_t* __restrict__ rows_out, int32_t* __restrict__ n_rows_out,
                                                     int32_t* __restrict__ runs_out) {
  const int qi = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const int64_t t = paged ? ctx_len[qi] - 1 : q_pos0 + qi;
  const int32_t* pt = paged ? page_table + qi * pt_stride : nullptr;
  const int n_sink = static_cast<int>(min64(S, t + 1));
  const int64_t win0 = max64(S, t - W + 1);
  const int n_win = static_cast<int>(max64(0, t - win0 + 1));
  const int n_sp = n_sparse[qi];
  const int n_tot = n_sink + n_sp + n_win;
  const int ld = S + Ksp + W;
  int breaks = emit_rows<kConvertThreads>(tid, S, W, Ksp, paged, kv_page, sparse_idx + static_cast<int64_t>(qi) * Ksp, n_sp, t,
                                         pt, rows_out + static_cast<int64_t>(qi) * ld, runs_out != nullptr);
  if (tid == 0) n_rows_out[qi] = n_tot;
  if (runs_out != nullptr) {
    __shared__ int sh[kConvertThreads / 32];
    breaks = __reduce_add_sync(0xffffffffu, breaks);
    if ((tid & 31) == 0) sh[tid >> 5] = breaks;
    __syncthreads();
    if (tid == 0) {
      int total = 0;
      for (int i = 0; i < kConvertThreads / 32; ++i) total += sh[i];
      int32_t* ro = runs_out + static_cast<int64_t>(qi) * 4;
      ro[0] = n_sink;
      ro[1] = n_sp;
      ro[2] = n_win;
      ro[3] = total;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// MinMax pooling (Eq. 13), contiguous caches: the coarse stage with per-dimension extrema of a sub-block in
// place of its mean.  max(q*a, q*b) with a >= b is q*a for q >= 0 and q*b for q < 0, so
// s~ = [max(q,0) | min(q,0)] . [k_max | k_min]: the Eq. 9 kernel's tile with rows of 2*d_I dims.
// ------------------------------------------------------------------------------------------------
template <bool E4M3>
__global__ void block_minmax_kernel(const uint8_t* __restrict__ k_idx, const float* __restrict__ k_scale,
                                    int64_t n_key, int DI, int B, __nv_bfloat16* __restrict__ kminmax) {
  const int U = DI / 8;  // 8 dims per thread
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t sub = gid / U;
  const int u = static_cast<int>(gid % U);
  if (sub * B >= n_key) return;
  const int64_t row0 = sub * B;
  const int cnt = static_cast<int>(min64(B, n_key - row0));
  float hi[8], lo[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    hi[j] = -INFINITY;
    lo[j] = INFINITY;
  }
  for (int r = 0; r < cnt; ++r) {
    const int64_t row = row0 + r;
    float v[8];
    if (E4M3) {
      const uint2 c = *reinterpret_cast<const uint2*>(k_idx + row * DI + u * 8);
      const float sc = k_scale[row];
      const uint32_t w[2] = {c.x, c.y};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(
            static_cast<__nv_fp8x2_storage_t>((w[j >> 1] >> ((j & 1) * 16)) & 0xffff), __NV_E4M3);
        const float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
        v[2 * j] = f.x * sc;
        v[2 * j + 1] = f.y * sc;
      }
    } else {
      const uint4 c = *reinterpret_cast<const uint4*>(k_idx + (row * DI + u * 8) * 2);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(h[j]);
        v[2 * j] = f.x;
        v[2 * j + 1] = f.y;
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      hi[j] = fmaxf(hi[j], v[j]);
      lo[j] = fminf(lo[j], v[j]);
    }
  }
  uint4 oh, ol;
  oh.x = pack_bf16(hi[0], hi[1]); oh.y = pack_bf16(hi[2], hi[3]); oh.z = pack_bf16(hi[4], hi[5]); oh.w = pack_bf16(hi[6], hi[7]);
  ol.x = pack_bf16(lo[0], lo[1]); ol.y = pack_bf16(lo[2], lo[3]); ol.z = pack_bf16(lo[4], lo[5]); ol.w = pack_bf16(lo[6], lo[7]);
  __nv_bfloat16* out = kminmax + sub * 2 * DI;
  *reinterpret_cast<uint4*>(out + u * 8) = oh;          // [k_max | k_min]
  *reinterpret_cast<uint4*>(out + DI + u * 8) = ol;
}

template <int HI, int DI>
struct CoarseMinMaxSmem {
  alignas(128) uint8_t a[kTileRows * DI * 4];     // 128 sub-blocks x [k_max | k_min]
  alignas(128) uint8_t q[2][HI * DI * 4];         // [q+ | q-] per head, two queries in flight
  float w[2][HI];
  float sub[kTileRows];
};

// One block = one tile of 128 sub-blocks x a group of queries (as coarse_score_kernel); a query's heads are split
// into positive and negative parts on their way into shared memory.
template <int HI, int DI>
__global__ void __launch_bounds__(kThreads) coarse_minmax_kernel(IndexArgs p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  auto& sm = *reinterpret_cast<CoarseMinMaxSmem<HI, DI>*>(smem_raw);
  constexpr int D2 = 2 * DI;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int spp = p.P / p.B;
  const int ppt = kTileRows / spp;
  const int64_t sub0 = static_cast<int64_t>(blockIdx.x) * kTileRows;
  const int64_t page0 = sub0 / spp;
  const int q_begin = blockIdx.y * kCoarseQG;
  const int q_end = min(p.n_query, q_begin + kCoarseQG);
  const int64_t n_key = p.n_key;
  // a query needs this tile iff the tile's first page is eligible and the coarse stage runs at all for it
  const int64_t t_need = max(page0 * p.P + p.W, (static_cast<int64_t>(p.M) + p.S / p.P) * p.P + p.W);
  if (p.q_pos0 + q_end - 1 < t_need) return;
  int q_first = q_begin;
  if (t_need - p.q_pos0 > q_begin) q_first = static_cast<int>(t_need - p.q_pos0);

  const int64_t n_sub = (n_key + p.B - 1) / p.B;
  {
    constexpr int U = D2 / 8;
    const uint8_t* km = reinterpret_cast<const uint8_t*>(p.kmean);
    for (int e = tid; e < kTileRows * U; e += kThreads) {
      const int r = e / U, u = e % U;
      const int64_t sub = sub0 + r;
      cp_async16(smem_u32(sm.a) + swz<D2 * 2>(r, u), km + (sub < n_sub ? sub : 0) * D2 * 2 + u * 16, sub < n_sub ? 16 : 0);
    }
    cp_async_commit();
  }
  constexpr int UQ = DI / 8;                       // 16-byte units of one head's query row
  constexpr int kPerThread = (HI * UQ + kThreads - 1) / kThreads;
  const uint8_t* qg = reinterpret_cast<const uint8_t*>(p.q_idx);
  auto load_q = [&](int qi, uint4 (&v)[kPerThread]) {
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
      const int e = tid + j * kThreads;
      v[j] = e < HI * UQ ? *reinterpret_cast<const uint4*>(qg + (static_cast<int64_t>(qi) * HI * UQ + e) * 16) : make_uint4(0, 0, 0, 0);
    }
  };
  auto store_q = [&](int qi, int buf, const uint4 (&v)[kPerThread]) {
    const __nv_bfloat162 zero = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
      const int e = tid + j * kThreads;
      if (e >= HI * UQ) continue;
      const int h = e / UQ, u = e % UQ;
      uint4 pos, neg;
      const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&v[j]);
      __nv_bfloat162* xp = reinterpret_cast<__nv_bfloat162*>(&pos);
      __nv_bfloat162* xn = reinterpret_cast<__nv_bfloat162*>(&neg);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        xp[i] = __hmax2(x[i], zero);
        xn[i] = __hmin2(x[i], zero);
      }
      *reinterpret_cast<uint4*>(sm.q[buf] + swz<D2 * 2>(h, u)) = pos;
      *reinterpret_cast<uint4*>(sm.q[buf] + swz<D2 * 2>(h, UQ + u)) = neg;
    }
    if (tid < HI) sm.w[buf][tid] = p.w[static_cast<int64_t>(qi) * HI + tid];
  };
  uint4 qv[kPerThread];
  load_q(q_first, qv);
  store_q(q_first, 0, qv);
  cp_async_wait<0>();
  __syncthreads();
  uint32_t a[D2 / 16][4];
  load_a_frags<D2>(a, smem_u32(sm.a));

  for (int qi = q_first; qi < q_end; ++qi) {
    const int buf = (qi - q_first) & 1;
    if (qi + 1 < q_end) load_q(qi + 1, qv);       // in flight during the scoring
    float s_lo, s_hi;
    score_16rows<HI, D2>(a, smem_u32(sm.q[buf]), sm.w[buf], s_lo, s_hi);
    if ((lane & 3) == 0) {
      sm.sub[16 * warp + (lane >> 2)] = s_lo;
      sm.sub[16 * warp + (lane >> 2) + 8] = s_hi;
    }
    if (qi + 1 < q_end) store_q(qi + 1, buf ^ 1, qv);   // the other buffer: last read one iteration ago, before a barrier
    __syncthreads();
    if (tid < ppt) {
      const int64_t page = page0 + tid;
      const int64_t hi = p.q_pos0 + qi - p.W;
      if (page * p.P <= hi) {
        float s = 0.f;
        for (int j = 0; j < spp; ++j) s += sm.sub[tid * spp + j];
        p.page_scores[static_cast<int64_t>(qi) * p.ps_ld + page] = s;
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// Decode-step cache maintenance: store the new token's indexer key (quantised for e4m3 caches), recompute the
// mean of its sub-block, copy the new rows of the attention caches.  One block per sequence, one thread per
// 8 key dims for the mean (same accumulation order and arithmetic as block_means_kernel).
// ------------------------------------------------------------------------------------------------
constexpr int kAppendThreads = 128;

__global__ void __launch_bounds__(kAppendThreads) append_kernel(AppendArgs a) {
  const int b = blockIdx.x, tid = threadIdx.x;
  const int DI = a.DI, U = DI / 8;
  pdl_wait();
  pdl_launch_dependents();
  const int64_t pos = a.ctx_len[b];
  const int64_t phys = a.page_table[b * a.pt_stride + pos / a.kv_page];
  const int64_t row = phys * a.kv_page + pos % a.kv_page;
  const __nv_bfloat16* kn = reinterpret_cast<const __nv_bfloat16*>(a.k_new) + static_cast<int64_t>(b) * DI;
  __shared__ float red[kAppendThreads / 32];
  __shared__ float s_scale;
  if (a.key_e4m3) {
    // per-token scale: amax / 448, then one code per dim
    float amax = 0.f;
    for (int d = tid; d < DI; d += kAppendThreads) amax = fmaxf(amax, fabsf(__bfloat162float(kn[d])));
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((tid & 31) == 0) red[tid >> 5] = amax;
    __syncthreads();
    if (tid == 0) {
      float m = 0.f;
      for (int i = 0; i < kAppendThreads / 32; ++i) m = fmaxf(m, red[i]);
      const float sc = m > 0.f ? __fdiv_rn(m, 448.0f) : 1.0f;
      s_scale = sc;
      a.k_scale[row] = sc;
    }
    __syncthreads();
    const float sc = s_scale;
    uint8_t* dst = reinterpret_cast<uint8_t*>(a.k_idx) + row * DI;
    for (int d = tid; d < DI; d += kAppendThreads)
      dst[d] = static_cast<uint8_t>(__nv_cvt_float_to_fp8(__fdiv_rn(__bfloat162float(kn[d]), sc), __NV_SATFINITE, __NV_E4M3));
  } else {
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.k_idx) + row * DI;
    for (int d = tid; d < DI; d += kAppendThreads) dst[d] = kn[d];
  }
  // attention caches of the group's layers
  for (int i = 0; i < a.n_kv; ++i) {
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a.kv_new[i]) + b * a.kv_row_bytes);
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(a.kv_pool[i]) + row * a.kv_row_bytes);
    for (int c = tid; c < a.kv_row_bytes / 16; c += kAppendThreads) dst[c] = src[c];
  }
  if (tid == 0 && a.ctx_len_out != nullptr) a.ctx_len_out[b] = static_cast<int32_t>(pos + 1);
  __syncthreads();   // the new key is in the pool (this block wrote it): the mean reads it back like any other row
  if (tid < U) {
    const int u = tid;
    const int64_t in_page = pos % a.kv_page;
    const int64_t pos0 = pos - pos % a.B;                  // first token of the sub-block (B divides kv_page)
    const int64_t row0 = row - (pos - pos0);
    const int cnt = static_cast<int>(pos - pos0 + 1);
    const int64_t out_row = phys * (a.kv_page / a.B) + in_page / a.B;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int r = 0; r < cnt; ++r) {
      const int64_t rr = row0 + r;
      if (a.key_e4m3) {
        const uint2 c = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint8_t*>(a.k_idx) + rr * DI + u * 8);
        const float sc = a.k_scale[rr];
        const uint32_t w[2] = {c.x, c.y};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(
              static_cast<__nv_fp8x2_storage_t>((w[j >> 1] >> ((j & 1) * 16)) & 0xffff), __NV_E4M3);
          const float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
          acc[2 * j] += f.x * sc;
          acc[2 * j + 1] += f.y * sc;
        }
      } else {
        const uint4 c = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a.k_idx) + (rr * DI + u * 8) * 2);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(h[j]);
          acc[2 * j] += f.x;
          acc[2 * j + 1] += f.y;
        }
      }
    }
    const float inv = static_cast<float>(cnt);
    uint4 o;
    o.x = pack_bf16(acc[0] / inv, acc[1] / inv);
    o.y = pack_bf16(acc[2] / inv, acc[3] / inv);
    o.z = pack_bf16(acc[4] / inv, acc[5] / inv);
    o.w = pack_bf16(acc[6] / inv, acc[7] / inv);
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(a.kmean) + out_row * DI + u * 8) = o;
  }
}

template <class K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
}

}  // namespace

bool index_shape_supported(int HI, int DI) { return (HI == 8 && DI == 64) || (HI == 64 && DI == 128); }

cudaError_t launch_block_means(int DI, int key_e4m3, int B, int kv_page, const void* k_idx, const float* k_scale,
                               int64_t n_key, const int32_t* page_table, int64_t pt_stride,
                               const int32_t* ctx_len, int batch, void* kmean, cudaStream_t st, int64_t* n_launch) {
  const int U = DI / 8;
  // paged: upper bound on sub-blocks per sequence is pt_stride * kv_page / B
  const int64_t n_sub = page_table ? pt_stride * kv_page / B : (n_key + B - 1) / B;
  if (n_sub == 0) return cudaSuccess;
  const int threads = 256;
  dim3 grid(static_cast<unsigned>((n_sub * U + threads - 1) / threads), page_table ? batch : 1);
  auto* kp = reinterpret_cast<const uint8_t*>(k_idx);
  auto* km = reinterpret_cast<__nv_bfloat16*>(kmean);
  if (key_e4m3)
    block_means_kernel<true><<<grid, threads, 0, st>>>(kp, k_scale, n_key, DI, B, kv_page, page_table, pt_stride, ctx_len, km);
  else
    block_means_kernel<false><<<grid, threads, 0, st>>>(kp, k_scale, n_key, DI, B, kv_page, page_table, pt_stride, ctx_len, km);
  ++*n_launch;
  return cudaGetLastError();
}

template <int HI, int DI>
static cudaError_t launch_coarse_t(const IndexArgs& a, int64_t n_key_max, cudaStream_t st, int64_t* n_launch) {
  const size_t smem = sizeof(CoarseSmem<HI, DI>);
  cudaError_t e = set_smem(coarse_score_kernel<HI, DI>, smem);
  if (e != cudaSuccess) return e;
  const int64_t n_sub = (n_key_max + a.B - 1) / a.B;
  const unsigned n_tiles = static_cast<unsigned>((n_sub + kTileRows - 1) / kTileRows);
  if (a.paged) {
    const size_t psmem = sizeof(CoarsePagedSmem<HI, DI>);
    e = set_smem(coarse_score_paged_kernel<HI, DI>, psmem);
    if (e != cudaSuccess) return e;
    dim3 pgrid((n_tiles + kCoarseTilesPerBlock - 1) / kCoarseTilesPerBlock, a.n_query);
    coarse_score_paged_kernel<HI, DI><<<pgrid, kThreads, psmem, st>>>(a);
    ++*n_launch;
    return cudaGetLastError();
  }
  dim3 grid(n_tiles, (a.n_query + kCoarseQG - 1) / kCoarseQG);
  coarse_score_kernel<HI, DI><<<grid, kThreads, smem, st>>>(a);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_coarse(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  // key tiles that any query can need: up to the largest cached length
  const int64_t n_key_max = a.paged ? a.pt_stride * a.P : a.n_key;
  if (coarse_paged_tc_supported(a)) return launch_coarse_paged_tc(a, st, n_launch);
  if (a.HI == 8 && a.DI == 64) return launch_coarse_t<8, 64>(a, n_key_max, st, n_launch);
  return launch_coarse_t<64, 128>(a, n_key_max, st, n_launch);
}

cudaError_t launch_append(const AppendArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.batch == 0) return cudaSuccess;
  const cudaError_t e = launch_pdl(append_kernel, dim3(a.batch), dim3(kAppendThreads), 0, st, a);
  ++*n_launch;
  return e;
}

cudaError_t launch_block_minmax(int DI, int key_e4m3, int B, const void* k_idx, const float* k_scale, int64_t n_key,
                                void* kminmax, cudaStream_t st, int64_t* n_launch) {
  const int U = DI / 8;
  const int64_t n_sub = (n_key + B - 1) / B;
  if (n_sub == 0) return cudaSuccess;
  const int threads = 256;
  const unsigned blocks = static_cast<unsigned>((n_sub * U + threads - 1) / threads);
  auto* kp = reinterpret_cast<const uint8_t*>(k_idx);
  auto* out = reinterpret_cast<__nv_bfloat16*>(kminmax);
  if (key_e4m3) block_minmax_kernel<true><<<blocks, threads, 0, st>>>(kp, k_scale, n_key, DI, B, out);
  else block_minmax_kernel<false><<<blocks, threads, 0, st>>>(kp, k_scale, n_key, DI, B, out);
  ++*n_launch;
  return cudaGetLastError();
}

template <int HI, int DI>
static cudaError_t launch_coarse_minmax_t(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  const size_t smem = sizeof(CoarseMinMaxSmem<HI, DI>);
  cudaError_t e = set_smem(coarse_minmax_kernel<HI, DI>, smem);
  if (e != cudaSuccess) return e;
  const int64_t n_sub = (a.n_key + a.B - 1) / a.B;
  dim3 grid(static_cast<unsigned>((n_sub + kTileRows - 1) / kTileRows), (a.n_query + kCoarseQG - 1) / kCoarseQG);
  coarse_minmax_kernel<HI, DI><<<grid, kThreads, smem, st>>>(a);
  ++*n_launch;
  return cudaGetLastError();
}

// a.kmean is the extrema cache [ceil(n_key/B), 2*DI]; contiguous caches only
cudaError_t launch_coarse_minmax(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  if (a.paged) return cudaErrorInvalidValue;
  if (a.HI == 8 && a.DI == 64) return launch_coarse_minmax_t<8, 64>(a, st, n_launch);
  return launch_coarse_minmax_t<64, 128>(a, st, n_launch);
}

template <int HI, int DI, bool E4M3>
static cudaError_t launch_fine_t(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  const size_t smem = sizeof(FineSmem<HI, DI>);
  cudaError_t e = set_smem(fine_select_kernel<HI, DI, E4M3>, smem);
  if (e != cudaSuccess) return e;
  const int parts = a.fine_parts > 1 ? a.fine_parts : 1;
  e = launch_pdl(fine_select_kernel<HI, DI, E4M3>, dim3(a.n_query, parts), dim3(kThreads), smem, st, a);
  if (e != cudaSuccess) return e;
  ++*n_launch;
  e = cudaGetLastError();
  if (e != cudaSuccess || parts == 1) return e;
  e = launch_pdl(fine_topk_kernel, dim3(a.n_query), dim3(kSelThreads), 0, st, a);
  if (e != cudaSuccess) return e;
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_fine_select(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  if (a.fine_cluster && fine_paged_tc_supported(a)) return launch_fine_paged_tc(a, a.sm_count, st, n_launch);
  if (a.fine_paged_tc && a.paged && a.fine_keys != nullptr && a.fine_pages != nullptr && paged_scores_tc_supported(a)) {
    // decode: page lists, then token scores of the listed pages on tcgen05, then the top-K_sparse with the cache rows
    cudaError_t e = launch_pdl(page_topm_paged_kernel, dim3(a.n_query), dim3(kSelThreads), 0, st, a);
    if (e != cudaSuccess) return e;
    ++*n_launch;
    e = launch_paged_scores_tc(a, 0, a.sm_count, st, n_launch);
    if (e != cudaSuccess) return e;
    e = launch_pdl(fine_topk_kernel, dim3(a.n_query), dim3(kSelThreads), 0, st, a);
    if (e != cudaSuccess) return e;
    ++*n_launch;
    return cudaGetLastError();
  }
  if (fine_tc_supported(a)) {
    cudaError_t e = launch_fine_select_tc(a, st, n_launch);
    if (e != cudaSuccess || a.fine_parts <= 1) return e;
    e = launch_pdl(fine_topk_kernel, dim3(a.n_query), dim3(kSelThreads), 0, st, a);
    if (e != cudaSuccess) return e;
    ++*n_launch;
    return cudaGetLastError();
  }
  if (a.HI == 8 && a.DI == 64)
    return a.key_e4m3 ? launch_fine_t<8, 64, true>(a, st, n_launch) : launch_fine_t<8, 64, false>(a, st, n_launch);
  return a.key_e4m3 ? launch_fine_t<64, 128, true>(a, st, n_launch) : launch_fine_t<64, 128, false>(a, st, n_launch);
}

cudaError_t launch_widen_e4m3(const void* codes, void* out_bf16, int64_t n_elems, cudaStream_t st, int64_t* n_launch) {
  const int64_t n_units = n_elems / 16;
  if (n_units == 0) return cudaSuccess;
  widen_e4m3_kernel<<<static_cast<unsigned>((n_units + 255) / 256), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(codes), reinterpret_cast<uint4*>(out_bf16), n_units);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_select(const float* scores, int64_t ld, const int32_t* cand_pos, const float* pos_scale,
                          int64_t q_pos0, int n_query, int64_t n_cand, int k, int apply_range, int S, int W,
                          int32_t* idx_out, int32_t* n_out, cudaStream_t st, int64_t* n_launch, const int32_t* ctx_len) {
  if (n_query == 0) return cudaSuccess;
  if (n_query <= kClusterRowsMax && n_cand >= kClusterMinRow) {
    // few long rows: a cluster of blocks per row
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(kClusterSel, static_cast<unsigned>(n_query), 1);
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = kClusterSel;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, select_cluster_kernel, scores, ld, cand_pos, pos_scale, q_pos0, n_cand, k,
                                             apply_range, S, W, idx_out, n_out, ctx_len);
    ++*n_launch;
    return e;
  }
  select_kernel<<<n_query, kSelThreads, 0, st>>>(scores, ld, cand_pos, pos_scale, q_pos0, n_cand, k, apply_range, S, W,
                                                 idx_out, n_out, ctx_len);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_convert(int S, int W, int Ksp, int paged, int kv_page, const int32_t* sparse_idx,
                           const int32_t* n_sparse, int64_t q_pos0, int n_query, const int32_t* page_table,
                           int64_t pt_stride, const int32_t* ctx_len, int32_t* rows_out, int32_t* n_rows_out,
                           int32_t* runs_out, cudaStream_t st, int64_t* n_launch) {
  if (n_query == 0) return cudaSuccess;
  const cudaError_t e = launch_pdl(convert_kernel, dim3(n_query), dim3(kConvertThreads), 0, st, S, W, Ksp, paged, kv_page, sparse_idx,
                                   n_sparse, q_pos0, page_table, pt_stride, ctx_len, rows_out, n_rows_out, runs_out);
  ++*n_launch;
  return e;
}

}  // namespace lsa
