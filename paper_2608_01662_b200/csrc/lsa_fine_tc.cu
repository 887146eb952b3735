// a2-a4 with the fine scores (Eq. 11) on the 5th-generation tensor cores, for the 64-head, 128-dim indexer.
//
// One thread block = one query (or one share of a query's candidate tiles when few queries must fill many SMs).
// After the page top-M (Eq. 10), the kept pages are scored in tiles of 128 candidate keys: keys are the M = 128
// rows of the MMA, the 64 heads its N, d_I = 128 its K (8 steps of M128 N64 K16 per tile):
//
//   warps 0-2   bring the tile's key rows into the 128B-swizzled K-major layout tcgen05.mma reads.  bf16 rows (bf16
//               caches, or e4m3 caches the caller widened once per call: k_wide) come by TMA, four 64-row boxes per
//               tile issued by one thread; without a widened copy the warps gather e4m3 codes and widen them in
//               registers (exact), the per-token scales riding along
//   warp 3      one thread issues the MMAs into one of two 64-column TMEM accumulators
//   warps 4-7   epilogue: tcgen05.ld, sum_j w_j * relu(acc_j) in-thread (one thread = one key), times the key's
//               scale, range check, order-preserving key into the candidate buffer
//
// and the candidate buffer then goes through the exact radix top-K_sparse (Eq. 12) with all eight warps.
#include "lsa_internal.h"
#include "lsa_select.cuh"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                 // candidate keys per tile
constexpr int kAtomA = kTile * 128;        // one 64-dim column block of a key tile
constexpr int kAtomQ = kHI * 128;          // one 64-dim column block of the query heads
constexpr int kFineThreads = 256;
constexpr int kLoadThreads = 96;           // warps 0-2
constexpr int kMaxSlotsTc = 4096;          // keep_pages * page
constexpr int kMaxPagesTc = 64;
constexpr uint32_t kTmemColsFine = 128;    // two accumulators of 64 columns

struct FineTcSmem {
  alignas(1024) uint8_t a[2][2][kAtomA];   // [buffer][column block][128 rows x 128 B]
  alignas(1024) uint8_t q[2][kAtomQ];      // [column block][64 rows x 128 B]
  float w[kHI];
  float scale[4][kTile];   // four deep: a tile's scales are read by the epilogue after its key buffer is already free
  uint32_t keys[kMaxSlotsTc];
  int32_t pages[kMaxPagesTc];
  SelectScratch sel;
  alignas(8) uint64_t k_full[2], k_empty[2], acc_full[2], acc_empty[2];
  uint32_t tmem_slot;
};

// TMA: key tiles are bf16 rows fetched through `map`; otherwise e4m3 codes gathered and widened by warps 0-2.
template <bool TMA>
__global__ void __launch_bounds__(kFineThreads, 2) fine_select_tc_kernel(const __grid_constant__ CUtensorMap map, IndexArgs p) {
  constexpr bool E4M3 = !TMA;   // the gather path exists for e4m3 codes only
  extern __shared__ uint8_t smem_raw[];
  FineTcSmem& sm = *reinterpret_cast<FineTcSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.x;
  const int part = blockIdx.y, n_parts = gridDim.y;
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
  if (hi < lo) {
    if (part != 0) return;
    if (n_parts > 1) p.fine_pages[qi * (kMaxPagesTc + 1) + kMaxPagesTc] = 0;
    for (int i = tid; i < p.Ksp; i += kFineThreads) out_idx[i] = -1;
    if (out_pages) for (int i = tid; i < p.M; i += kFineThreads) out_pages[i] = -1;
    if (tid == 0) p.n_sparse[qi] = 0;
    return;
  }
  if (tc::status_raised(p.status)) return;   // an earlier block of this launch gave up on a wait

  // query heads (K-major, 128B swizzle) and head weights: asynchronous copies that land during the page selection
  {
    const uint8_t* qg = reinterpret_cast<const uint8_t*>(p.q_idx) + static_cast<int64_t>(qi) * kHI * kDI * 2;
#pragma unroll
    for (int k = 0; k < kHI * 16 / kFineThreads; ++k) {
      const int e = tid + k * kFineThreads, r = e >> 4, c = e & 15;
      cp_async16(smem_u32(sm.q[c >> 3]) + r * 128 + (((c & 7) ^ (r & 7)) << 4), qg + e * 16, 16);
    }
    if (tid < kHI / 4) cp_async16(smem_u32(&sm.w[tid * 4]), p.w + static_cast<int64_t>(qi) * kHI + tid * 4, 16);
    cp_async_commit();
  }

  // ---- a2: pages that survive the coarse stage
  const int p0 = static_cast<int>(lo / p.P), p1 = static_cast<int>(hi / p.P);
  const int nE = p1 - p0 + 1;
  int nP;
  if (p.hi_enable && nE > p.M) {
    const float* ps = p.page_scores + static_cast<int64_t>(qi) * p.ps_ld + p0;
    if (nE <= kMaxSlotsTc) {
      for (int i = tid; i < nE; i += kFineThreads) sm.keys[i] = score_key(ps[i]);
      __syncthreads();
      nP = block_select_topk([&](int i) { return sm.keys[i]; }, [&](int i) { return p0 + i; }, nE, p.M, sm.pages, sm.sel);
    } else {
      nP = block_select_topk<0, true>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M, sm.pages,
                             sm.sel);
    }
  } else {
    nP = nE;  // the host guarantees nE * P <= kMaxSlotsTc here
    for (int i = tid; i < nP; i += kFineThreads) sm.pages[i] = p0 + i;
  }

  // ---- set-up of the tile pipeline
  if (tid == 0) {
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.k_full[b]), TMA ? 1 : kLoadThreads);
      tc::mbar_init(smem_u32(&sm.k_empty[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
    }
    tc::fence_mbar_init();
  }
  if (warp == 3) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsFine);
    tc::tmem_relinquish();
  }
  cp_async_wait<0>();   // query heads and weights, requested before the page selection
  tc::fence_proxy_async();
  tc::fence_before_sync();
  __syncthreads();   // pages, q, w, barriers and the TMEM base are visible
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;

  if (out_pages && part == 0) for (int i = tid; i < p.M; i += kFineThreads) out_pages[i] = i < nP ? sm.pages[i] : -1;
  if (n_parts > 1 && part == 0) {
    int32_t* fp = p.fine_pages + qi * (kMaxPagesTc + 1);
    for (int i = tid; i < nP; i += kFineThreads) fp[i] = sm.pages[i];
    if (tid == 0) fp[kMaxPagesTc] = nP;
  }
  const int n_slots = nP * p.P;
  const int n_tiles_all = (n_slots + kTile - 1) / kTile;
  const int tiles_per = (n_tiles_all + n_parts - 1) / n_parts;
  const int tile0 = part * tiles_per;
  const int n_tiles = max(0, min(n_tiles_all, tile0 + tiles_per) - tile0);
  const int pshift = 31 - __clz(p.P);
  auto slot_pos = [&](int c) -> int64_t { return static_cast<int64_t>(sm.pages[c >> pshift]) * p.P + (c & (p.P - 1)); };
  auto phys_row = [&](int64_t pos) -> int64_t {
    return p.paged ? static_cast<int64_t>(pt[pos >> pshift]) * p.P + (pos & (p.P - 1)) : pos;
  };

  if (TMA && warp < 3) {
    // ================= TMA producers: lane 0 of warps 0 and 1 takes the boxes of one 64-row half of every tile each
    // (an issued TMA copy costs its thread 200-300 cycles: four boxes per tile from one thread were a good part of a
    // tile's time).  Warp 0 arrives on the barrier with the byte count of the whole tile; a box of warp 1 that completes
    // before that only makes the count negative for a moment =================
    if (lane == 0 && warp < 2) {
      const int h = warp;
      for (int i = 0; i < n_tiles; ++i) {
        const int b = i & 1;
        if (!tc::mbar_wait(smem_u32(&sm.k_empty[b]), ((i >> 1) & 1) ^ 1, p.status)) break;
        if (h == 0) tc::mbar_expect_tx(smem_u32(&sm.k_full[b]), 2 * kAtomA);
        // 64 consecutive slots lie in one page; rows past the cache read as zero
        const int c = (tile0 + i) * kTile + 64 * h;
        const int row = c < n_slots ? static_cast<int>(slot_pos(c)) : static_cast<int>(n_key);
#pragma unroll
        for (int cb = 0; cb < 2; ++cb)
          tc::tma_load_2d(smem_u32(sm.a[b][cb]) + h * 64 * 128, &map, cb * 64, row, smem_u32(&sm.k_full[b]));
      }
    }
  } else if (warp < 3) {
    // ================= gather warps =================
    // Each thread owns whole key rows (rows tid and tid + 96 of the tile): all 16-byte loads of a row are in flight
    // together, then the row is widened and stored.  Rows of one page are consecutive in memory, so a warp's loads
    // cover contiguous 128- or 256-byte segments.
    const uint8_t* kbase = reinterpret_cast<const uint8_t*>(p.k_idx);
    constexpr int kUnitsPerRow = E4M3 ? 8 : 16;          // 16-byte units of a key row in global memory
    constexpr int kRowBytes = E4M3 ? kDI : kDI * 2;
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i & 1;
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.k_empty[b]), ((i >> 1) & 1) ^ 1, p.status))) break;
      const int c0 = (tile0 + i) * kTile;
      for (int r = tid; r < kTile; r += kLoadThreads) {
        const int c = c0 + r;
        int64_t row = -1;
        if (c < n_slots) {
          const int64_t pos = slot_pos(c);
          if (pos < n_key) row = phys_row(pos);
        }
        uint4 v[kUnitsPerRow];
#pragma unroll
        for (int u = 0; u < kUnitsPerRow; ++u)
          v[u] = row >= 0 ? *reinterpret_cast<const uint4*>(kbase + row * kRowBytes + u * 16) : make_uint4(0, 0, 0, 0);
        if constexpr (E4M3) sm.scale[i & 3][r] = row >= 0 ? p.k_scale[row] : 0.f;
#pragma unroll
        for (int u = 0; u < kUnitsPerRow; ++u) {
          if constexpr (E4M3) {
            uint4 lo16, hi16;   // 16 codes -> dims 16u .. 16u+15 = bf16 chunks 2u, 2u+1 of the row
            e4m3x16_to_bf16(v[u], lo16, hi16);
            uint8_t* dst = sm.a[b][u >> 2] + r * 128;
            *reinterpret_cast<uint4*>(dst + ((((2 * u) & 7) ^ (r & 7)) << 4)) = lo16;
            *reinterpret_cast<uint4*>(dst + ((((2 * u + 1) & 7) ^ (r & 7)) << 4)) = hi16;
          } else {
            *reinterpret_cast<uint4*>(sm.a[b][u >> 3] + r * 128 + (((u & 7) ^ (r & 7)) << 4)) = v[u];
          }
        }
      }
      tc::fence_proxy_async();
      tc::mbar_arrive(smem_u32(&sm.k_full[b]));
    }
  } else if (warp == 3) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.a), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int b = i & 1;
        ok = tc::mbar_wait(smem_u32(&sm.k_full[b]), (i >> 1) & 1, p.status) &&
             tc::mbar_wait(smem_u32(&sm.acc_empty[b]), ((i >> 1) & 1) ^ 1, p.status);
        if (!ok) break;
        tc::fence_after_sync();
        const uint32_t d = tmem_base + b * kHI;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // 16-dim step: column block ks/4, 32-byte slice ks%4
          tc::umma_ss(d, tc::desc_advance(da0, b * 2 * kAtomA + (ks >> 2) * kAtomA + (ks & 3) * 32),
                      tc::desc_advance(dq0, (ks >> 2) * kAtomQ + (ks & 3) * 32), idesc, ks != 0);
        tc::umma_commit(smem_u32(&sm.k_empty[b]));
        tc::umma_commit(smem_u32(&sm.acc_full[b]));
      }
    }
  } else {
    // ================= epilogue warps =================
    const int quarter = warp & 3;          // warps 4-7 own TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;     // key row of the tile
    bool ok = true;
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int b = i & 1;
      const int c = (tile0 + i) * kTile + r;
      const int64_t pos = c < n_slots ? slot_pos(c) : -1;
      const bool cand = pos >= lo && pos <= hi;
      float sc = 1.f;
      if (TMA && p.key_e4m3 && cand) sc = p.k_scale[pos];   // in flight while the tile's MMAs run
      ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[b]), (i >> 1) & 1, p.status));
      if (!ok) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + b * kHI, v);
      tc::tmem_ld_wait();
      if (!TMA) sc = sm.scale[i & 3][r];   // read before the accumulator is handed back
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
      if (c < n_slots) sm.keys[c] = cand ? score_key((a0 + a1) * sc) : 0u;
    }
  }
  tc::fence_before_sync();
  __syncthreads();   // every tile of this block is scored
  if (warp == 3) tc::tmem_dealloc(tmem_base, kTmemColsFine);

  if (n_parts > 1) {
    // hand this block's share of the candidate keys to the top-K kernel
    uint32_t* fk = p.fine_keys + static_cast<int64_t>(qi) * kMaxSlotsTc;
    const int c0 = tile0 * kTile, c1 = min(n_slots, (tile0 + n_tiles) * kTile);
    for (int c = c0 + tid; c < c1; c += kFineThreads) fk[c] = sm.keys[c];
    return;
  }
  const int n_sel = block_select_topk([&](int i) { return sm.keys[i]; },
                                      [&](int i) { return static_cast<int>(slot_pos(i)); }, n_slots, p.Ksp, out_idx,
                                      sm.sel);
  if (tid == 0) p.n_sparse[qi] = n_sel;
}

template <bool TMA>
cudaError_t launch_t(const IndexArgs& a, const CUtensorMap& map, cudaStream_t st, int64_t* n_launch) {
  const size_t smem = sizeof(FineTcSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(fine_select_tc_kernel<TMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int parts = a.fine_parts > 1 ? a.fine_parts : 1;
  fine_select_tc_kernel<TMA><<<dim3(a.n_query, parts), kFineThreads, smem, st>>>(map, a);
  ++*n_launch;
  return cudaGetLastError();
}

// bf16 key rows the TMA path can read: the cache itself, or the widened copy of an e4m3 cache
const void* bf16_rows(const IndexArgs& a) { return a.key_e4m3 ? a.k_wide : a.k_idx; }

}  // namespace

// Contiguous caches only: a paged decode step has few tiles per block, where the pipeline set-up outweighs the gain.
// bf16 caches need the 16-byte alignment of a TMA source.
bool fine_tc_supported(const IndexArgs& a) {
  if (a.HI != kHI || a.DI != kDI || a.paged) return false;
  const void* rows = bf16_rows(a);
  if (rows != nullptr) return (reinterpret_cast<uintptr_t>(rows) & 15u) == 0 && tma_available();
  return a.key_e4m3 != 0;
}

// Scoring blocks only; with fine_parts > 1 the caller follows up with the top-K kernel of lsa_index.cu.
cudaError_t launch_fine_select_tc(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  CUtensorMap map{};
  const void* rows = bf16_rows(a);
  if (rows == nullptr) return launch_t<false>(a, map, st, n_launch);
  if (!make_map_bf16_128(&map, rows, static_cast<uint64_t>(a.n_key), 64)) return cudaErrorInvalidValue;
  return launch_t<true>(a, map, st, n_launch);
}

}  // namespace lsa
