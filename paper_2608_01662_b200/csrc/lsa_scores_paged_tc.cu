// Token scores (Eq. 1 / Eq. 11) over pages of a paged cache on the 5th-generation tensor cores, 64-head / 128-dim
// indexer.  Two users:
//
//   fine stage of the hierarchy (a3, decode): the pages the coarse stage kept (lists written by page_topm_kernel)
//     -> order-preserving keys of the candidate slots, from which fine_topk_kernel takes the top-K_sparse;
//   flat indexer (Eq. 7, hi_enable = 0): every page that holds a position of the scoring range
//     -> fp32 scores per position, from which the row selection takes the top-K_sparse.
//
// A cache page (64 tokens) is one contiguous piece of the key pool, so a tile (two pages = the M = 128 rows of the MMA;
// the 64 heads are its N, d_I = 128 its K) is fetched with two bulk copies, plus two for the per-token scales of an
// e4m3 cache.  Sequences differ in length, so the tiles of all sequences form one list and each block (one per SM)
// takes an equal contiguous share of it.  Inside a block:
//
//   warp 0       producer.  Page numbers come from two dependent look-ups (page list, page table); the 32 lanes do
//                them for 32 tiles at a time, lane 0 then issues the bulk copies into a ring of raw tiles deep enough
//                for the few microseconds a fetch from a multi-GB pool takes, and the TMA loads of a sequence's query
//                heads (two slots) when the share crosses into the next sequence
//   warps 8-15   widen: a landed raw tile -> the 128B-swizzled K-major bf16 operand (e4m3 -> bf16 is exact; bf16 caches
//                are just re-laid out), per-token scales set aside for the epilogue
//   warp 1       one thread issues 8 x tcgen05.mma (M128 N64 K16) per tile into one of two TMEM accumulators
//   warps 4-7    epilogue: one thread = one token: sum_j w_j relu(acc_j), times the token's scale, out
#include "lsa_internal.h"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                  // tokens per tile: two cache pages
constexpr int kPageTok = 64;
constexpr int kAtomA = kTile * 128;         // one 64-dim column block of a tile
constexpr int kAtomQ = kHI * 128;
constexpr int kThreadsPs = 512;
constexpr int kWidenThreads = 256;          // warps 8-15
constexpr int kMaxBatchPs = 1024;
constexpr int kMaxPagesPs = 64;             // page-list pitch is kMaxPagesPs + 1 (the count comes last)
constexpr int kMaxSlotsPs = 4096;
constexpr uint32_t kTmemColsPs = 128;       // two accumulators of 64 columns

template <bool E4M3>
struct PsSmem {
  static constexpr int kRawTileBytes = E4M3 ? kTile * kDI : kTile * kDI * 2;
  static constexpr int kRawSlots = E4M3 ? 6 : 3;
  alignas(1024) uint8_t a[2][2][kAtomA];      // operand: [buffer][64-dim half][128 rows x 128 B]
  alignas(1024) uint8_t q[2][2][kAtomQ];      // [query slot][64-dim half]
  alignas(128) uint8_t raw[kRawSlots][kRawTileBytes];
  alignas(16) float raw_scale[kRawSlots][kTile];
  float scale[4][kTile];   // four deep: the epilogue reads a tile's scales after its operand buffer is free again
  float w[2][kHI];
  int32_t ntile[kMaxBatchPs];   // per sequence: tiles, pages and first page of its list, cached length
  int32_t npage[kMaxBatchPs];
  int32_t page0[kMaxBatchPs];
  int32_t ctx[kMaxBatchPs];
  alignas(8) uint64_t raw_full[6], raw_empty[6], a_full[2], a_empty[2], acc_full[2], acc_empty[2], q_full[2], q_empty[2];
  uint32_t tmem_slot;
  int red[kThreadsPs / 32];
  int first_seq, first_tile;
};

struct PsShape {
  int S, W, flat;
};

// Pages a sequence of `ctx` cached tokens contributes.  Flat: the pages that hold a position of [S, ctx-1-W];
// otherwise the length of its page list.
__device__ __forceinline__ int pages_of(int ctx, const PsShape& sh, const int32_t* fine_pages, int seq, int* p0) {
  const int hi = ctx - 1 - sh.W;
  *p0 = sh.S / kPageTok;
  if (hi < sh.S) return 0;
  if (sh.flat) return hi / kPageTok - *p0 + 1;
  return fine_pages[seq * (kMaxPagesPs + 1) + kMaxPagesPs];
}

struct PsWalker {
  int seq, tile, n_in_seq;
  __device__ __forceinline__ void start(const int32_t* ntile, int s, int tl) {
    seq = s;
    tile = tl;
    n_in_seq = ntile[s];
  }
  // returns true when the next tile belongs to another sequence
  __device__ __forceinline__ bool next(const int32_t* ntile, int batch) {
    if (++tile < n_in_seq) return false;
    tile = 0;
    do {
      ++seq;
      n_in_seq = seq < batch ? ntile[seq] : 1;   // past the end: only reached after a block's last tile
    } while (n_in_seq == 0);
    return true;
  }
};

// global -> shared bulk copy; completion is counted in bytes on `bar`.  Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <bool E4M3>
__global__ void __launch_bounds__(kThreadsPs, 1)
paged_scores_tc_kernel(const __grid_constant__ CUtensorMap map_q, IndexArgs p, int flat) {
  using Smem = PsSmem<E4M3>;
  constexpr int kRawSlots = Smem::kRawSlots;
  constexpr int kRowBytes = E4M3 ? kDI : kDI * 2;            // a token's key in the pool
  constexpr int kPageBytes = kPageTok * kRowBytes;
  extern __shared__ uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int batch = p.n_query;
  PsShape sh;
  sh.S = p.S; sh.W = p.W; sh.flat = flat;
  if (tc::status_raised(p.status)) return;
  pdl_wait();                 // page lists and cached lengths come from earlier kernels of the stream
  pdl_launch_dependents();

  // ---- this block's share of the tile list
  int my_tiles = 0;
  for (int s = tid; s < batch; s += kThreadsPs) {
    int p0;
    const int c = p.ctx_len[s];
    const int np = pages_of(c, sh, p.fine_pages, s, &p0);
    sm.ctx[s] = c;
    sm.npage[s] = np;
    sm.page0[s] = p0;
    sm.ntile[s] = (np + 1) / 2;
    my_tiles += (np + 1) / 2;
  }
  my_tiles = __reduce_add_sync(0xffffffffu, my_tiles);
  if (lane == 0) sm.red[warp] = my_tiles;
  __syncthreads();
  int total = 0;
  for (int i = 0; i < kThreadsPs / 32; ++i) total += sm.red[i];
  const int g0 = static_cast<int>(static_cast<int64_t>(total) * blockIdx.x / gridDim.x);
  const int g1 = static_cast<int>(static_cast<int64_t>(total) * (blockIdx.x + 1) / gridDim.x);
  const int n_tiles = g1 - g0;
  if (n_tiles <= 0) return;
  if (warp == 0) {
    // sequence and tile that hold list position g0: a warp-wide scan, 32 sequences per round
    int base = 0, found_seq = -1, found_tile = 0;
    for (int s0 = 0; s0 < batch && found_seq < 0; s0 += 32) {
      const int n = s0 + lane < batch ? sm.ntile[s0 + lane] : 0;
      int incl = n;
      for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
      }
      const bool here = g0 >= base + incl - n && g0 < base + incl;
      const unsigned m = __ballot_sync(0xffffffffu, here);
      if (m) {
        const int l = __ffs(m) - 1;
        found_seq = s0 + l;
        found_tile = g0 - (base + __shfl_sync(0xffffffffu, incl - n, l));
      }
      base += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
      sm.first_seq = found_seq;
      sm.first_tile = found_tile;
    }
  }

  if (tid == 0) {
    for (int s = 0; s < kRawSlots; ++s) {
      tc::mbar_init(smem_u32(&sm.raw_full[s]), 1);
      tc::mbar_init(smem_u32(&sm.raw_empty[s]), kWidenThreads / 32);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.a_full[b]), kWidenThreads / 32);
      tc::mbar_init(smem_u32(&sm.a_empty[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
      tc::mbar_init(smem_u32(&sm.q_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.q_empty[b]), 5);   // the MMA thread's commit and the four epilogue warps
    }
    tc::fence_mbar_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsPs);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;
  PsWalker wk;
  wk.start(sm.ntile, sm.first_seq, sm.first_tile);

  // logical pages of tile `tile` of sequence `seq` (-1: the tile has no second page)
  auto tile_pages = [&](int seq, int tile, int* lp0, int* lp1) {
    const int n_pages = sm.npage[seq];
    if (flat) {
      *lp0 = sm.page0[seq] + 2 * tile;
      *lp1 = 2 * tile + 1 < n_pages ? *lp0 + 1 : -1;
    } else {
      const int32_t* list = p.fine_pages + seq * (kMaxPagesPs + 1);
      *lp0 = list[2 * tile];
      *lp1 = 2 * tile + 1 < n_pages ? list[2 * tile + 1] : -1;
    }
  };

  if (warp == 0) {
    // ================= producer =================
    const uint8_t* kbase = reinterpret_cast<const uint8_t*>(p.k_idx);
    int n_q = 0;
    int prev_seq = -1;
    bool alive = true;
    for (int base = 0; base < n_tiles && alive; base += 32) {
      // lane l: physical pages of tile base + l
      PsWalker mine = wk;
      for (int s = 0; s < lane; ++s) mine.next(sm.ntile, batch);
      int my_seq = -1, ph0 = -1, ph1 = -1;
      if (base + lane < n_tiles) {
        int lp0, lp1;
        my_seq = mine.seq;
        tile_pages(mine.seq, mine.tile, &lp0, &lp1);
        const int32_t* pt = p.page_table + static_cast<int64_t>(mine.seq) * p.pt_stride;
        ph0 = pt[lp0];
        ph1 = lp1 >= 0 ? pt[lp1] : -1;
      }
      for (int s = 0; s < 32; ++s) wk.next(sm.ntile, batch);   // (walking past the share's end is harmless)
      const int n_here = min(32, n_tiles - base);
      for (int j = 0; j < n_here && alive; ++j) {
        const int i = base + j;
        const int seq = __shfl_sync(0xffffffffu, my_seq, j);
        const int f0 = __shfl_sync(0xffffffffu, ph0, j), f1 = __shfl_sync(0xffffffffu, ph1, j);
        bool ok = true;
        if (seq != prev_seq) {
          // query heads and head weights of this sequence into slot n_q & 1
          const int slot = n_q & 1;
          if (lane == 0) ok = tc::mbar_wait(smem_u32(&sm.q_empty[slot]), ((n_q >> 1) & 1) ^ 1, p.status);
          if (!__shfl_sync(0xffffffffu, ok, 0)) { alive = false; break; }
          sm.w[slot][lane] = p.w[static_cast<int64_t>(seq) * kHI + lane];
          sm.w[slot][lane + 32] = p.w[static_cast<int64_t>(seq) * kHI + lane + 32];
          __syncwarp();
          if (lane == 0) {
            tc::mbar_expect_tx(smem_u32(&sm.q_full[slot]), 2 * kAtomQ);
            tc::tma_load_2d(smem_u32(sm.q[slot][0]), &map_q, 0, seq * kHI, smem_u32(&sm.q_full[slot]));
            tc::tma_load_2d(smem_u32(sm.q[slot][1]), &map_q, 64, seq * kHI, smem_u32(&sm.q_full[slot]));
          }
          ++n_q;
          prev_seq = seq;
        }
        if (lane == 0) {
          const int s = i % kRawSlots;
          ok = tc::mbar_wait(smem_u32(&sm.raw_empty[s]), ((i / kRawSlots) & 1) ^ 1, p.status);
          if (ok) {
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
        if (!__shfl_sync(0xffffffffu, ok, 0)) alive = false;
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.a), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      int n_q = 0;
      bool new_seq = true;
      for (int i = 0; i < n_tiles; ++i) {
        const int b = i & 1;
        if (new_seq) {
          if (!tc::mbar_wait(smem_u32(&sm.q_full[n_q & 1]), (n_q >> 1) & 1, p.status)) break;
          ++n_q;
        }
        const int slot = (n_q - 1) & 1;
        new_seq = wk.next(sm.ntile, batch);
        if (!tc::mbar_wait(smem_u32(&sm.a_full[b]), (i >> 1) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[b]), ((i >> 1) & 1) ^ 1, p.status))
          break;
        tc::fence_after_sync();
        const uint32_t d = tmem_base + b * kHI;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // 16-dim step: column block ks/4, 32-byte slice ks%4
          tc::umma_ss(d, tc::desc_advance(da0, b * 2 * kAtomA + (ks >> 2) * kAtomA + (ks & 3) * 32),
                      tc::desc_advance(dq0, slot * 2 * kAtomQ + (ks >> 2) * kAtomQ + (ks & 3) * 32), idesc, ks != 0);
        tc::umma_commit(smem_u32(&sm.a_empty[b]));
        tc::umma_commit(smem_u32(&sm.acc_full[b]));
        if (new_seq || i + 1 == n_tiles) tc::umma_commit(smem_u32(&sm.q_empty[slot]));   // last tile of its sequence here
      }
    }
  } else if (warp >= 8) {
    // ================= widen warps =================
    const int wt = tid - 256;   // 0..255
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kRawSlots, b = i & 1;
      if (!tc::mbar_wait(smem_u32(&sm.raw_full[s]), (i / kRawSlots) & 1, p.status) ||
          !tc::mbar_wait(smem_u32(&sm.a_empty[b]), ((i >> 1) & 1) ^ 1, p.status))
        break;
      if constexpr (E4M3) {
        if (wt < kTile) sm.scale[i & 3][wt] = sm.raw_scale[s][wt];
#pragma unroll
        for (int j = 0; j < kTile * 8 / kWidenThreads; ++j) {   // 16 codes -> dims 16u .. 16u+15 = bf16 chunks 2u, 2u+1 of the row
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
    int n_q = 0;
    bool new_seq = true;
    // the page of this row's token is looked up one tile ahead (a page-list entry comes from L2)
    int lp_next;
    {
      int lp0, lp1;
      tile_pages(wk.seq, wk.tile, &lp0, &lp1);
      lp_next = r < kPageTok ? lp0 : lp1;
    }
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i & 1;
      if (new_seq) {
        // the head weights of the slot were stored before the arrival on q_full
        if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.q_full[n_q & 1]), (n_q >> 1) & 1, p.status))) break;
        ++n_q;
      }
      const int slot = (n_q - 1) & 1;
      const int seq = wk.seq, tile = wk.tile;
      new_seq = wk.next(sm.ntile, batch);
      const int lp = lp_next;
      if (i + 1 < n_tiles) {
        int lp0, lp1;
        tile_pages(wk.seq, wk.tile, &lp0, &lp1);
        lp_next = r < kPageTok ? lp0 : lp1;
      }
      const int ctx = sm.ctx[seq];
      const int64_t pos = lp >= 0 ? static_cast<int64_t>(lp) * kPageTok + (r & (kPageTok - 1)) : -1;
      const bool cand = pos >= sh.S && pos <= static_cast<int64_t>(ctx) - 1 - sh.W;
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
      const float4* w4 = reinterpret_cast<const float4*>(sm.w[slot]);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float4 ww = w4[j];
        a0 = fmaf(ww.x, fmaxf(__uint_as_float(v[4 * j + 0]), 0.f), a0);
        a1 = fmaf(ww.y, fmaxf(__uint_as_float(v[4 * j + 1]), 0.f), a1);
        a0 = fmaf(ww.z, fmaxf(__uint_as_float(v[4 * j + 2]), 0.f), a0);
        a1 = fmaf(ww.w, fmaxf(__uint_as_float(v[4 * j + 3]), 0.f), a1);
      }
      if (new_seq || i + 1 == n_tiles) {   // done with this sequence's head weights
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(smem_u32(&sm.q_empty[slot]));
      }
      const float score = (a0 + a1) * sc;
      if (flat) {
        if (cand) p.page_scores[static_cast<int64_t>(seq) * p.ps_ld + pos] = score;
      } else if (lp >= 0) {
        p.fine_keys[static_cast<int64_t>(seq) * kMaxSlotsPs + tile * kTile + r] = cand ? score_key(score) : 0u;
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemColsPs);
}

}  // namespace

// Paged caches with 64-token pages (kv_page = P = 64), the 64-head / 128-dim indexer, 16-byte aligned pools.
bool paged_scores_tc_supported(const IndexArgs& a) {
  return a.paged && a.HI == kHI && a.DI == kDI && a.P == kPageTok && a.n_query <= kMaxBatchPs &&
         (reinterpret_cast<uintptr_t>(a.k_idx) & 15u) == 0 && (reinterpret_cast<uintptr_t>(a.q_idx) & 15u) == 0 &&
         (!a.key_e4m3 || (reinterpret_cast<uintptr_t>(a.k_scale) & 15u) == 0) && tma_available();
}

// flat = 0: keys of the candidate slots of the page lists in a.fine_pages -> a.fine_keys;
// flat = 1: scores of every position of the scoring range -> a.page_scores [n_query, ps_ld] (one column per position).
cudaError_t launch_paged_scores_tc(const IndexArgs& a, int flat, int sm_count, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  CUtensorMap map_q;
  if (!make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kHI)) return cudaErrorInvalidValue;
  const int64_t max_tiles = flat ? (a.pt_stride + 1) / 2 * a.n_query : static_cast<int64_t>(kMaxPagesPs / 2) * a.n_query;
  int64_t blocks = sm_count > 0 ? sm_count : 148;
  if (blocks > max_tiles) blocks = max_tiles;
  if (blocks < 1) blocks = 1;
  cudaError_t e;
  if (a.key_e4m3) {
    const size_t smem = sizeof(PsSmem<true>) + 1024;
    e = cudaFuncSetAttribute(paged_scores_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = launch_pdl(paged_scores_tc_kernel<true>, dim3(static_cast<unsigned>(blocks)), dim3(kThreadsPs), smem, st, map_q, a, flat);
  } else {
    const size_t smem = sizeof(PsSmem<false>) + 1024;
    e = cudaFuncSetAttribute(paged_scores_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = launch_pdl(paged_scores_tc_kernel<false>, dim3(static_cast<unsigned>(blocks)), dim3(kThreadsPs), smem, st, map_q, a, flat);
  }
  ++*n_launch;
  return e;
}

}  // namespace lsa
