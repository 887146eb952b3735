// a2-a3 for recall budgets beyond what one thread block can keep in shared memory (M * P > 4096 candidate
// tokens per query; the paper's own operating point recalls 128K tokens, Sec. 5 "Recall budget"), contiguous caches,
// 64-head / 128-dim indexer.
//
//   page_topm_kernel        a2: one block per query selects the M eligible pages with the largest coarse score
//                           (Eq. 10; the exact radix select, reading the scores from global memory) into a page list
//   fine_scores_tc_kernel   a3: the fine scores (Eq. 11) of the listed pages on tcgen05 as in lsa_fine_tc.cu (TMA key
//                           tiles of 128 tokens from the bf16 rows, M128 N64 K16, epilogue sum_j w_j relu(.) x scale),
//                           but the scores go to global memory as order-preserving keys (0 = not a candidate): a block
//                           covers a run of a query's tiles, several blocks share a query
//
//   select_keys_kernel      a4: the exact radix top-K_sparse over each query's keys; a slot's position comes from the page
//                           list, so only the keys (4 bytes per candidate) travel through memory
#include "lsa_internal.h"
#include "lsa_select.cuh"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;
constexpr int kAtomA = kTile * 128;
constexpr int kAtomQ = kHI * 128;
constexpr int kThreadsBig = 192;           // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int kStagesBig = 2;               // two blocks per SM
constexpr int kTilesPerBlockBig = 32;
constexpr uint32_t kTmemColsBig = 128;

// ---- a2
__global__ void __launch_bounds__(kSelThreads) page_topm_kernel(IndexArgs p, int32_t* __restrict__ pages_ws,
                                                                int32_t* __restrict__ n_pages_ws) {
  __shared__ SelectScratch sc;
  const int qi = blockIdx.x, tid = threadIdx.x;
  const int64_t t = p.q_pos0 + qi;
  const int64_t lo = p.S, hi = t - p.W;
  int32_t* out = pages_ws + static_cast<int64_t>(qi) * p.M;
  int32_t* out_user = p.pages_out ? p.pages_out + static_cast<int64_t>(qi) * p.M : nullptr;
  int nP = 0;
  if (hi >= lo) {
    const int p0 = static_cast<int>(lo / p.P), p1 = static_cast<int>(hi / p.P);
    const int nE = p1 - p0 + 1;
    if (p.hi_enable && nE > p.M) {
      const float* ps = p.page_scores + static_cast<int64_t>(qi) * p.ps_ld + p0;
      nP = block_select_topk<0, true>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M, out, sc);
    } else {
      nP = nE;   // the host sized M so that every eligible page fits the list when the hierarchy is off
      for (int i = tid; i < p.M; i += kSelThreads) out[i] = i < nP ? p0 + i : -1;
    }
  } else {
    for (int i = tid; i < p.M; i += kSelThreads) out[i] = -1;
  }
  __syncthreads();
  if (out_user) for (int i = tid; i < p.M; i += kSelThreads) out_user[i] = out[i];
  if (tid == 0) n_pages_ws[qi] = nP;
}

// ---- a3
struct FineBigSmem {
  alignas(1024) uint8_t a[kStagesBig][2][kAtomA];
  alignas(1024) uint8_t q[2][kAtomQ];
  float w[kHI];
  alignas(8) uint64_t full[kStagesBig], empty[kStagesBig], acc_full[2], acc_empty[2];
  uint32_t tmem_slot;
};

__global__ void __launch_bounds__(kThreadsBig, 2)
fine_scores_tc_kernel(const __grid_constant__ CUtensorMap map, IndexArgs p, const int32_t* __restrict__ pages_ws,
                      const int32_t* __restrict__ n_pages_ws, uint32_t* __restrict__ keys, int64_t ld) {
  extern __shared__ uint8_t smem_raw[];
  FineBigSmem& sm = *reinterpret_cast<FineBigSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.x;
  const int64_t t = p.q_pos0 + qi;
  const int64_t lo = p.S, hi = t - p.W;
  const int pshift = 31 - __clz(p.P);
  const int nP = n_pages_ws[qi];
  const int n_slots = nP << pshift;
  const int tile_begin = blockIdx.y * kTilesPerBlockBig;
  const int tiles_all = static_cast<int>(ld / kTile);                   // the whole row, listed pages or not
  const int tile_end = min(tiles_all, tile_begin + kTilesPerBlockBig);
  const int tiles_live = min(tile_end, (n_slots + kTile - 1) / kTile);  // tiles that hold listed pages
  const int32_t* pages = pages_ws + static_cast<int64_t>(qi) * p.M;
  uint32_t* krow = keys + static_cast<int64_t>(qi) * ld;
  // slots past the listed pages: marked absent for the top-K
  for (int c = max(tile_begin, tiles_live) * kTile + tid; c < tile_end * kTile; c += kThreadsBig) krow[c] = 0u;
  const int n_tiles = tiles_live - tile_begin;
  if (n_tiles <= 0) return;
  if (tc::status_raised(p.status)) return;

  if (tid == 0) {
    for (int s = 0; s < kStagesBig; ++s) {
      tc::mbar_init(smem_u32(&sm.full[s]), 1);
      tc::mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
    }
    tc::fence_mbar_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsBig);
    tc::tmem_relinquish();
  }
  {
    const uint8_t* qg = reinterpret_cast<const uint8_t*>(p.q_idx) + static_cast<int64_t>(qi) * kHI * kDI * 2;
    for (int e = tid; e < kHI * 16; e += kThreadsBig) {
      const int r = e >> 4, c = e & 15;
      cp_async16(smem_u32(sm.q[c >> 3]) + r * 128 + (((c & 7) ^ (r & 7)) << 4), qg + e * 16, 16);
    }
    if (tid < kHI / 4) cp_async16(smem_u32(&sm.w[tid * 4]), p.w + static_cast<int64_t>(qi) * kHI + tid * 4, 16);
    cp_async_commit();
    cp_async_wait<0>();
  }
  tc::fence_proxy_async();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;
  auto slot_pos = [&](int c) -> int64_t { return (static_cast<int64_t>(pages[c >> pshift]) << pshift) + (c & (p.P - 1)); };

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kStagesBig;
        if (!tc::mbar_wait(smem_u32(&sm.empty[s]), ((i / kStagesBig) & 1) ^ 1, p.status)) break;
        tc::mbar_expect_tx(smem_u32(&sm.full[s]), 2 * kAtomA);
#pragma unroll
        for (int h = 0; h < 2; ++h) {   // 64 consecutive slots lie in one page; rows past the cache read as zero
          const int c = (tile_begin + i) * kTile + 64 * h;
          const int row = c < n_slots ? static_cast<int>(slot_pos(c)) : static_cast<int>(p.n_key);
#pragma unroll
          for (int cb = 0; cb < 2; ++cb)
            tc::tma_load_2d(smem_u32(sm.a[s][cb]) + h * 64 * 128, &map, cb * 64, row, smem_u32(&sm.full[s]));
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.a), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kStagesBig, b = i & 1;
        if (!tc::mbar_wait(smem_u32(&sm.full[s]), (i / kStagesBig) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[b]), ((i >> 1) & 1) ^ 1, p.status))
          break;
        tc::fence_after_sync();
        const uint32_t d = tmem_base + b * kHI;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          tc::umma_ss(d, tc::desc_advance(da0, s * 2 * kAtomA + (ks >> 2) * kAtomA + (ks & 3) * 32),
                      tc::desc_advance(dq0, (ks >> 2) * kAtomQ + (ks & 3) * 32), idesc, ks != 0);
        tc::umma_commit(smem_u32(&sm.empty[s]));
        tc::umma_commit(smem_u32(&sm.acc_full[b]));
      }
    }
  } else {
    // ================= epilogue warps =================
    const int quarter = warp & 3;          // warps 2-5 own TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i & 1;
      const int c = (tile_begin + i) * kTile + r;
      const int64_t pos = c < n_slots ? slot_pos(c) : -1;
      const bool cand = pos >= lo && pos <= hi;
      float sc = 1.f;
      if (p.key_e4m3 && cand) sc = p.k_scale[pos];   // in flight while the tile's MMAs run
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[b]), (i >> 1) & 1, p.status))) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + b * kHI, v);
      tc::tmem_ld_wait();
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(smem_u32(&sm.acc_empty[b]));
      float a0 = 0.f, a1 = 0.f;
      const float4* w4 = reinterpret_cast<const float4*>(sm.w);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float4 ww = w4[j];
        a0 = fmaf(ww.x, fmaxf(__uint_as_float(v[4 * j + 0]), 0.f), a0);
        a1 = fmaf(ww.y, fmaxf(__uint_as_float(v[4 * j + 1]), 0.f), a1);
        a0 = fmaf(ww.z, fmaxf(__uint_as_float(v[4 * j + 2]), 0.f), a0);
        a1 = fmaf(ww.w, fmaxf(__uint_as_float(v[4 * j + 3]), 0.f), a1);
      }
      krow[c] = cand ? score_key((a0 + a1) * sc) : 0u;   // order-preserving key; outside the scoring range: absent
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemColsBig);
}

// ---- a4 over the keys of a query's listed pages: slot c of the row is token pages[c / P] * P + c % P
__global__ void __launch_bounds__(kSelThreads) select_keys_kernel(IndexArgs p, const int32_t* __restrict__ pages_ws,
                                                                  const int32_t* __restrict__ n_pages_ws,
                                                                  const uint32_t* __restrict__ keys, int64_t ld) {
  __shared__ SelectScratch sc;
  __shared__ int32_t pages[1024];
  const int qi = blockIdx.x, tid = threadIdx.x;
  const int pshift = 31 - __clz(p.P);
  const int nP = n_pages_ws[qi];
  const bool cached = p.M <= 1024;
  const int32_t* pg = pages_ws + static_cast<int64_t>(qi) * p.M;
  if (cached) {
    for (int i = tid; i < nP; i += kSelThreads) pages[i] = pg[i];
    __syncthreads();
    pg = pages;
  }
  const uint32_t* krow = keys + static_cast<int64_t>(qi) * ld;
  const int n_sel = block_select_topk([&](int i) { return krow[i]; },
                                      [&](int i) { return (pg[i >> pshift] << pshift) + (i & (p.P - 1)); }, nP << pshift, p.Ksp,
                                      p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp, sc);
  if (tid == 0) p.n_sparse[qi] = n_sel;
}

}  // namespace

// Contiguous cache, 64-head / 128-dim indexer, bf16 rows reachable by TMA (the cache itself or the widened copy).
bool fine_big_supported(const IndexArgs& a) {
  const void* rows = a.key_e4m3 ? a.k_wide : a.k_idx;
  return !a.paged && a.HI == kHI && a.DI == kDI && rows != nullptr && (reinterpret_cast<uintptr_t>(rows) & 15u) == 0 &&
         tma_available();
}

// pages_ws int32 [n_query, M], n_pages_ws int32 [n_query], keys uint32 [n_query, M * P]; three launches: page lists,
// fine scores as order-preserving keys, top-K_sparse
cudaError_t launch_fine_big(const IndexArgs& a, int32_t* pages_ws, int32_t* n_pages_ws, uint32_t* keys, cudaStream_t st,
                            int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  page_topm_kernel<<<a.n_query, kSelThreads, 0, st>>>(a, pages_ws, n_pages_ws);
  ++*n_launch;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  CUtensorMap map;
  const void* rows = a.key_e4m3 ? a.k_wide : a.k_idx;
  if (!make_map_bf16_128(&map, rows, static_cast<uint64_t>(a.n_key), 64)) return cudaErrorInvalidValue;
  const size_t smem = sizeof(FineBigSmem) + 1024;
  e = cudaFuncSetAttribute(fine_scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int64_t ld = static_cast<int64_t>(a.M) * a.P;
  const unsigned parts = static_cast<unsigned>((ld / kTile + kTilesPerBlockBig - 1) / kTilesPerBlockBig);
  fine_scores_tc_kernel<<<dim3(a.n_query, parts), kThreadsBig, smem, st>>>(map, a, pages_ws, n_pages_ws, keys, ld);
  ++*n_launch;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  select_keys_kernel<<<a.n_query, kSelThreads, 0, st>>>(a, pages_ws, n_pages_ws, keys, ld);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace lsa
