// Fine stage of the hierarchical indexer on paged caches (a2-a5 in decode) as one kernel: top-M pages of a sequence
// (Eq. 10), token scores of the kept pages on the 5th-generation tensor cores (Eq. 11), top-K_sparse (Eq. 12) and
// the sequence's cache rows for the attention kernels (streaming-aware conversion).  64-head / 128-dim indexer,
// 64-token cache pages (a cache page is a selection page), up to 64 kept pages.
//
// A sequence is owned by a thread-block cluster of one or two blocks.  Every block of the cluster selects the pages
// (the same list in each: no exchange needed), takes its share of the list's tiles (two pages = the M = 128 rows of an
// MMA; the 64 heads are N, d_I = 128 is K) and scores them; the candidate keys of all blocks land in the shared memory
// of the cluster's first block (remote stores of 4 bytes per token), which takes the top-K and writes the results.
// The scores never leave the SMs.
//
// Inside a block, after the page selection (threads 0-255):
//   warp 0       producer: one bulk copy per page (a page is one contiguous piece of the key pool) and one for its
//                per-token scales (e4m3 caches) into a ring of raw tiles
//   warps 8-15   widen: a landed raw tile -> the 128B-swizzled K-major bf16 operand (e4m3 -> bf16 is exact)
//   warps 1, 2   one thread of each issues 8 x tcgen05.mma (M128 N64 K16) per tile, warp 1 for the even tiles and
//                warp 2 for the odd ones, each into its own TMEM accumulator
//   warps 4-7    epilogue: one thread = one token: sum_j w_j relu(acc_j), times the token's scale, as an
//                order-preserving key into the first block's candidate array
// The query heads arrive by TMA before the dependency wait (they are an input of the call, not a product of the
// coarse kernel that precedes this one in the stream).
#include "lsa_internal.h"
#include "lsa_select.cuh"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                  // tokens per tile: two cache pages
constexpr int kPageTok = 64;
constexpr int kAtomA = kTile * 128;         // one 64-dim column block of a tile
constexpr int kAtomQ = kHI * 128;
constexpr int kThreadsFp = 512;
constexpr int kWidenThreads = 256;          // warps 8-15
constexpr int kMaxPagesFp = 64;
constexpr int kMaxSlotsFp = kMaxPagesFp * kPageTok;
constexpr uint32_t kTmemColsFp = 128;       // two accumulators of 64 columns
constexpr int kSelBar = 1;                  // named barrier of threads 0-255 (the selections)

template <bool E4M3>
struct FpSmem {
  static constexpr int kRawTileBytes = E4M3 ? kTile * kDI : kTile * kDI * 2;
  static constexpr int kRawSlots = E4M3 ? 6 : 3;
  alignas(1024) uint8_t a[2][2][kAtomA];      // operand: [buffer][64-dim half][128 rows x 128 B]
  alignas(1024) uint8_t q[2][kAtomQ];         // query heads: [64-dim half][64 rows x 128 B]
  // ring of raw tiles; before the first copy it holds the keys of the page scores (up to kMaxSlotsFp of them)
  alignas(128) uint8_t raw[kRawSlots][kRawTileBytes];
  alignas(16) float raw_scale[kRawSlots][kTile];
  float scale[4][kTile];   // four deep: the epilogue reads a tile's scales after its operand buffer is free again
  float w[kHI];
  uint32_t keys[kMaxSlotsFp];   // candidate keys of the whole cluster (used in the first block only)
  int32_t pages[kMaxPagesFp];   // kept pages, ascending
  int32_t phys[kMaxPagesFp];    // their places in the pool
  SelectScratch sel;
  alignas(8) uint64_t raw_full[6], raw_empty[6], a_full[2], acc_full[2], acc_empty[2], q_full;
  uint32_t tmem_slot;
};
static_assert(sizeof(FpSmem<true>) + 1024 <= 227 * 1024 && sizeof(FpSmem<false>) + 1024 <= 227 * 1024, "shared memory");
static_assert(FpSmem<true>::kRawSlots * FpSmem<true>::kRawTileBytes >= kMaxSlotsFp * 4, "page keys fit the ring");

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
// Address of this block's shared-memory location `addr` in the block of rank `rank` of the cluster.
__device__ __forceinline__ uint32_t smem_of_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void store_cluster_u32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// global -> shared bulk copy; completion is counted in bytes on `bar`.  Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// a4 + a5 for one sequence (all threads of the cluster's first block): top-K_sparse of the candidate keys by threads
// 0-255, ascending positions, written both as positions (sparse_idx) and as the cache rows the attention kernels read
// (the pages' places in the pool are at hand: no page-table look-up per row); then the sink and window rows and the
// padding of the row list by everybody.  Row list: [sink | sparse | window | -1 ...], S + Ksp + W entries.
// Inlined: the selection's scratch and the key array must be known to be shared memory (generic atomics are slow).
__device__ __forceinline__ void finish_sequence(const IndexArgs& p, const uint32_t* keys, const int32_t* pages, const int32_t* phys,
                                             SelectScratch& sel, int n_slots, int qi, int64_t t) {
  const int tid = threadIdx.x;
  const int ld = p.S + p.Ksp + p.W;
  const int n_sink = static_cast<int>(min64(p.S, t + 1));
  int32_t* rows = p.rows_out != nullptr ? p.rows_out + static_cast<int64_t>(qi) * ld : nullptr;
  if (tid < kSelThreads) {
    int32_t* out_idx = p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp;
    const int n_sel = block_select_topk_emit<kSelBar>(
        [&](int i) { return keys[i]; },
        [&](int r, int i) {
          out_idx[r] = pages[i >> 6] * kPageTok + (i & (kPageTok - 1));
          if (rows != nullptr) rows[n_sink + r] = phys[i >> 6] * kPageTok + (i & (kPageTok - 1));
        },
        [&](int r) { out_idx[r] = -1; }, n_slots, p.Ksp, sel);
    if (tid == 0) {
      p.n_sparse[qi] = n_sel;
      sel.n_valid = static_cast<uint32_t>(n_sel);
    }
  }
  __syncthreads();
  if (rows == nullptr) return;
  const int n_sel = static_cast<int>(sel.n_valid);
  const int64_t win0 = max64(p.S, t - p.W + 1);
  const int n_win = static_cast<int>(max64(0, t - win0 + 1));
  const int32_t* pt = p.page_table + static_cast<int64_t>(qi) * p.pt_stride;
  // everything but the sparse part: ld - n_sel entries
  for (int j = tid; j < ld - n_sel; j += kThreadsFp) {
    int32_t r = -1;
    int at = j;
    if (j < n_sink) {
      r = static_cast<int32_t>(static_cast<int64_t>(pt[j >> 6]) * kPageTok + (j & (kPageTok - 1)));
    } else {
      at = j + n_sel;
      if (j - n_sink < n_win) {
        const int64_t pos = win0 + (j - n_sink);
        r = static_cast<int32_t>(static_cast<int64_t>(pt[pos >> 6]) * kPageTok + (pos & (kPageTok - 1)));
      }
    }
    rows[at] = r;
  }
  if (tid == 0) p.n_rows_out[qi] = n_sink + n_sel + n_win;
}

template <bool E4M3>
__global__ void __launch_bounds__(kThreadsFp, 1)
fine_paged_tc_kernel(const __grid_constant__ CUtensorMap map_q, IndexArgs p) {
  using Smem = FpSmem<E4M3>;
  constexpr int kRawSlots = Smem::kRawSlots;
  constexpr int kRowBytes = E4M3 ? kDI : kDI * 2;            // a token's key in the pool
  constexpr int kPageBytes = kPageTok * kRowBytes;
  extern __shared__ uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.y;
  const uint32_t rank = cluster_rank(), n_rank = cluster_size();
  // The cluster barrier has no time limit: every path below reaches both of its phases, also after a failed wait.
  cluster_arrive();   // phase 1: "this block runs" (its shared memory may be written from now on)
  const bool live = !tc::status_raised(p.status);

  if (tid == 0) {
    for (int s = 0; s < kRawSlots; ++s) {
      tc::mbar_init(smem_u32(&sm.raw_full[s]), 1);
      tc::mbar_init(smem_u32(&sm.raw_empty[s]), kWidenThreads / 32);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.a_full[b]), kWidenThreads / 32);
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
    }
    tc::mbar_init(smem_u32(&sm.q_full), 1);
    tc::fence_mbar_init();
    if (live) {
      tc::mbar_expect_tx(smem_u32(&sm.q_full), 2 * kAtomQ);
      tc::tma_load_2d(smem_u32(sm.q[0]), &map_q, 0, qi * kHI, smem_u32(&sm.q_full));
      tc::tma_load_2d(smem_u32(sm.q[1]), &map_q, 64, qi * kHI, smem_u32(&sm.q_full));
    }
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsFp);
    tc::tmem_relinquish();
  }
  if (tid < kHI) sm.w[tid] = p.w[static_cast<int64_t>(qi) * kHI + tid];
  pdl_wait();                 // the page scores come from the coarse kernel
  pdl_launch_dependents();

  // ---- a2: the pages of this sequence that survive the coarse stage, ascending (every block of the cluster)
  const int64_t t = static_cast<int64_t>(p.ctx_len[qi]) - 1;
  const int64_t lo = p.S, hi = t - p.W;
  const int32_t* pt = p.page_table + static_cast<int64_t>(qi) * p.pt_stride;
  int nP = 0;
  if (tid < kSelThreads) {
    if (live && hi >= lo) {
      const int p0 = static_cast<int>(lo / kPageTok), p1 = static_cast<int>(hi / kPageTok);
      const int nE = p1 - p0 + 1;
      if (p.hi_enable && nE > p.M) {
        const float* ps = p.page_scores + static_cast<int64_t>(qi) * p.ps_ld + p0;
        if (nE <= kMaxSlotsFp) {
          uint32_t* pk = reinterpret_cast<uint32_t*>(sm.raw);
          for (int i0 = tid; i0 < nE; i0 += 8 * kSelThreads) {   // eight loads in flight per thread
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = i0 + u * kSelThreads < nE ? ps[i0 + u * kSelThreads] : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u)
              if (i0 + u * kSelThreads < nE) pk[i0 + u * kSelThreads] = score_key(v[u]);
          }
          select_sync<kSelBar>();
          nP = block_select_topk<kSelBar>([&](int i) { return pk[i]; }, [&](int i) { return p0 + i; }, nE, p.M, sm.pages, sm.sel);
          tc::fence_proxy_async();   // the ring is handed to the bulk copies
        } else {
          nP = block_select_topk<kSelBar>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M,
                                          sm.pages, sm.sel);
        }
      } else {
        nP = nE;   // the host guarantees nE <= kMaxPagesFp here
        for (int i = tid; i < nP; i += kSelThreads) sm.pages[i] = p0 + i;
        select_sync<kSelBar>();
      }
      for (int i = tid; i < nP; i += kSelThreads) sm.phys[i] = pt[sm.pages[i]];
    }
    if (rank == 0 && p.pages_out != nullptr)
      for (int i = tid; i < p.M; i += kSelThreads) p.pages_out[static_cast<int64_t>(qi) * p.M + i] = i < nP ? sm.pages[i] : -1;
    if (tid == 0) sm.sel.n_valid = static_cast<uint32_t>(nP);   // for the other half of the block
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  nP = static_cast<int>(sm.sel.n_valid);
  const uint32_t tmem_base = sm.tmem_slot;
  const int n_slots = nP * kPageTok;
  const int n_tiles_all = (nP + 1) / 2;
  const int tiles_per = (n_tiles_all + static_cast<int>(n_rank) - 1) / static_cast<int>(n_rank);
  const int tile0 = static_cast<int>(rank) * tiles_per;
  const int n_tiles = max(0, min(n_tiles_all, tile0 + tiles_per) - tile0);
  cluster_wait();   // phase 1 complete: every block of the cluster runs

  if (warp == 0) {
    // ================= producer =================
    if (lane == 0) {
      const uint8_t* kbase = reinterpret_cast<const uint8_t*>(p.k_idx);
      for (int i = 0; i < n_tiles; ++i) {
        const int tl = tile0 + i;
        const int f0 = sm.phys[2 * tl];
        const int f1 = 2 * tl + 1 < nP ? sm.phys[2 * tl + 1] : -1;
        const int s = i % kRawSlots;
        if (!tc::mbar_wait(smem_u32(&sm.raw_empty[s]), ((i / kRawSlots) & 1) ^ 1, p.status)) break;
        const uint32_t bar = smem_u32(&sm.raw_full[s]);
        const uint32_t per_page = kPageBytes + (E4M3 ? kPageTok * 4 : 0);
        tc::mbar_expect_tx(bar, f1 >= 0 ? 2 * per_page : per_page);
        bulk_load(smem_u32(sm.raw[s]), kbase + static_cast<int64_t>(f0) * kPageBytes, kPageBytes, bar);
        if (E4M3) bulk_load(smem_u32(sm.raw_scale[s]), p.k_scale + static_cast<int64_t>(f0) * kPageTok, kPageTok * 4, bar);
        if (f1 >= 0) {
          bulk_load(smem_u32(sm.raw[s]) + kPageBytes, kbase + static_cast<int64_t>(f1) * kPageBytes, kPageBytes, bar);
          if (E4M3)
            bulk_load(smem_u32(&sm.raw_scale[s][kPageTok]), p.k_scale + static_cast<int64_t>(f1) * kPageTok, kPageTok * 4, bar);
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ================= MMA issuers: warp 1 takes the even tiles (operand buffer and accumulator 0), warp 2 the odd
    // ones; one thread issues an MMA every 55-90 cycles, two keep the pipe busy =================
    const int b = warp - 1;
    if (lane == 0 && n_tiles > b) {
      constexpr uint32_t idesc = tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.a[b]), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      uint64_t da[8], dq[8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {   // 16-dim step: column block ks/4, 32-byte slice ks%4
        da[ks] = tc::desc_advance(da0, (ks >> 2) * kAtomA + (ks & 3) * 32);
        dq[ks] = tc::desc_advance(dq0, (ks >> 2) * kAtomQ + (ks & 3) * 32);
      }
      const uint32_t d = tmem_base + b * kHI;
      bool ok = tc::mbar_wait(smem_u32(&sm.q_full), 0, p.status);
      for (int i = b; i < n_tiles && ok; i += 2) {
        if (!tc::mbar_wait(smem_u32(&sm.a_full[b]), (i >> 1) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[b]), ((i >> 1) & 1) ^ 1, p.status))
          break;
        tc::fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) tc::umma_ss(d, da[ks], dq[ks], idesc, ks != 0);
        tc::umma_commit(smem_u32(&sm.acc_full[b]));   // accumulator ready = operand buffer free again
      }
    }
  } else if (warp >= 8) {
    // ================= widen warps =================
    const int wt = tid - 256;   // 0..255
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kRawSlots, b = i & 1;
      if (!tc::mbar_wait(smem_u32(&sm.raw_full[s]), (i / kRawSlots) & 1, p.status) ||
          !tc::mbar_wait(smem_u32(&sm.acc_full[b]), ((i >> 1) & 1) ^ 1, p.status))   // MMAs of tile i - 2 complete
        break;
      if constexpr (E4M3) {
        if (wt < kTile) sm.scale[i & 3][wt] = sm.raw_scale[s][wt];
#pragma unroll
        for (int j = 0; j < kTile * 8 / kWidenThreads; ++j) {   // 16 codes -> dims 16u .. 16u+15 = 16-byte chunks 2u, 2u+1 of the row
          const int e = wt + j * kWidenThreads, r = e >> 3, u = e & 7;
          const uint4 c = *reinterpret_cast<const uint4*>(sm.raw[s] + e * 16);
          uint4 lo16, hi16;
          e4m3x16_to_bf16(c, lo16, hi16);
          uint8_t* dst = sm.a[b][u >> 2] + r * 128;
          *reinterpret_cast<uint4*>(dst + ((((2 * u) & 7) ^ (r & 7)) << 4)) = lo16;
          *reinterpret_cast<uint4*>(dst + ((((2 * u + 1) & 7) ^ (r & 7)) << 4)) = hi16;
        }
      } else {
#pragma unroll
        for (int j = 0; j < kTile * 16 / kWidenThreads; ++j) {
          const int e = wt + j * kWidenThreads, r = e >> 4, u = e & 15;
          *reinterpret_cast<uint4*>(sm.a[b][u >> 3] + r * 128 + (((u & 7) ^ (r & 7)) << 4)) =
              *reinterpret_cast<const uint4*>(sm.raw[s] + e * 16);
        }
      }
      tc::fence_proxy_async();
      __syncwarp();
      if (lane == 0) {   // one arrival per warp: 256 arrivals on one barrier are 256 serialised shared-memory operations
        tc::mbar_arrive(smem_u32(&sm.a_full[b]));
        tc::mbar_arrive(smem_u32(&sm.raw_empty[s]));
      }
    }
  } else if (warp >= 4) {
    // ================= epilogue warps =================
    const int quarter = warp & 3;          // warps 4-7 own TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;     // token row of the tile
    const uint32_t keys0 = smem_of_rank(smem_u32(sm.keys), 0);
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i & 1;
      const int c = (tile0 + i) * kTile + r;   // candidate slot
      int64_t pos = -1;
      if (c < n_slots) pos = static_cast<int64_t>(sm.pages[c >> 6]) * kPageTok + (c & (kPageTok - 1));
      const bool cand = pos >= lo && pos <= hi;
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[b]), (i >> 1) & 1, p.status))) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + b * kHI, v);
      tc::tmem_ld_wait();
      const float sc = E4M3 ? sm.scale[i & 3][r] : 1.f;   // read before the accumulator is handed back
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
      if (c < n_slots) store_cluster_u32(keys0 + static_cast<uint32_t>(c) * 4u, cand ? score_key((a0 + a1) * sc) : 0u);
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemColsFp);
  cluster_arrive();   // phase 2: this block's keys are in the first block's shared memory
  cluster_wait();
  if (rank != 0) return;
  finish_sequence(p, sm.keys, sm.pages, sm.phys, sm.sel, tc::status_raised(p.status) ? 0 : n_slots, qi, t);
}

}  // namespace

// Paged caches with 64-token pages (kv_page = P = 64), the 64-head / 128-dim indexer, at most 64 kept pages, 16-byte
// aligned pools.
bool fine_paged_tc_supported(const IndexArgs& a) {
  return a.paged && a.HI == kHI && a.DI == kDI && a.P == kPageTok && a.M <= kMaxPagesFp && a.Ksp <= kMaxSlotsFp &&
         (reinterpret_cast<uintptr_t>(a.k_idx) & 15u) == 0 && (reinterpret_cast<uintptr_t>(a.q_idx) & 15u) == 0 &&
         (!a.key_e4m3 || (reinterpret_cast<uintptr_t>(a.k_scale) & 15u) == 0) && tma_available();
}

// One cluster per sequence: two blocks while all clusters are resident at once, else one.
cudaError_t launch_fine_paged_tc(const IndexArgs& a, int sm_count, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  CUtensorMap map_q;
  if (!make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kHI)) return cudaErrorInvalidValue;
  const int sms = sm_count > 0 ? sm_count : 148;
  const unsigned n_rank = 2 * a.n_query <= sms ? 2u : 1u;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(n_rank, static_cast<unsigned>(a.n_query), 1);
  cfg.blockDim = dim3(kThreadsFp);
  cfg.stream = st;
  cudaLaunchAttribute attr[2]{};
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_rank;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol.wait in the kernel
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e;
  if (a.key_e4m3) {
    cfg.dynamicSmemBytes = sizeof(FpSmem<true>) + 1024;
    e = cudaFuncSetAttribute(fine_paged_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(cfg.dynamicSmemBytes));
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, fine_paged_tc_kernel<true>, map_q, a);
  } else {
    cfg.dynamicSmemBytes = sizeof(FpSmem<false>) + 1024;
    e = cudaFuncSetAttribute(fine_paged_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(cfg.dynamicSmemBytes));
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, fine_paged_tc_kernel<false>, map_q, a);
  }
  ++*n_launch;
  return e;
}

}  // namespace lsa
