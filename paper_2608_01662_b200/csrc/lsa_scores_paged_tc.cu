// Token scores (Eq. 1 / Eq. 11) over pages of a paged cache on the 5th-generation tensor cores, 64-head / 128-dim
// indexer.  Two users:
//
//   fine stage of the hierarchy (a3, decode): the pages the coarse stage kept (lists written by page_topm_kernel)
//     -> order-preserving keys of the candidate slots, from which fine_topk_kernel takes the top-K_sparse;
//   flat indexer (Eq. 7, hi_enable = 0): every page that holds a position of the scoring range
//     -> fp32 scores per position, from which the row selection takes the top-K_sparse.
//
// A cache page (64 tokens) is one TMA box: it lands in the 128B-swizzled K-major layout the MMA reads, and goes from
// the pool to the tensor cores untouched.  bf16 cache: kind::f16 MMAs against the bf16 query heads (8 x M128 N64 K16
// per tile of two pages).  e4m3 cache: the codes are the A operand of kind::f8f6f4 MMAs as they are, the query heads
// the B operand as three e5m2 planes that accumulate into one accumulator (12 x M128 N64 K32; see e5m2_head_shift /
// split_e5m2x16 in lsa_common.cuh: every product exact, the head's power-of-two scale folded into its weight).
// Sequences differ in length, so the tiles of all sequences form one list and each block (one per SM) takes an equal
// contiguous share of it.  Inside a block (16 warps; tile i of the share belongs to the producer, the issuer and the
// epilogue set of its parity, so that every ring slot and accumulator has one thread on each side of its barriers):
//
//   warps 0, 1   producers.  Page numbers come from two dependent look-ups (page list, page table); the 32 lanes do
//                them for 32 tiles at a time, lane 0 then issues its tiles' copies into a ring deep enough for the
//                few microseconds a fetch from a multi-GB pool takes: a TMA box per page (two for bf16) and a
//                256-byte bulk copy of the page's per-token scales (e4m3).  An issued copy costs its thread 200-300
//                cycles, hence two producers
//   warps 2, 3   one thread of each issues the MMAs of its tiles into accumulator i % 4 of TMEM
//   warps 4-7 / 8-11   epilogue of the even / odd tiles: one thread = one token: sum_j w_j relu(acc_j), times the
//                token's scale, out
//   warps 12-15  the query heads of the share's next sequence into the other of two slots: e5m2 planes built from
//                the bf16 heads (e4m3 cache) or a TMA load (bf16 cache), and the head weights
#include "lsa_internal.h"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                  // tokens per tile: two cache pages
constexpr int kPageTok = 64;
constexpr int kAtom = kTile * 128;          // 128 rows x 128 B
constexpr int kAtomQ = kHI * 128;
constexpr int kThreadsPs = 512;
constexpr int kQThreads = 128;              // warps 12-15
constexpr int kQBar = 2;                    // their named barrier
constexpr int kMaxBatchPs = 1024;
constexpr int kMaxPagesPs = 64;             // page-list pitch is kMaxPagesPs + 1 (the count comes last)
constexpr int kMaxSlotsPs = 4096;
constexpr uint32_t kTmemColsPs = 256;       // four accumulators of 64 columns

template <bool E4M3>
struct PsSmem {
  static constexpr int kRowBytes = E4M3 ? kDI : kDI * 2;         // a token's key in the pool
  static constexpr int kTileBytes = kTile * kRowBytes;           // e4m3: [128 rows x 128 B]; bf16: [64-dim half][128 rows x 128 B]
  static constexpr int kSlots = E4M3 ? 8 : 4;                    // 128 KB of key tiles in flight
  static constexpr int kQBytes = E4M3 ? 3 * kAtomQ : 2 * kAtomQ; // three e5m2 planes | two 64-dim halves, [64 heads x 128 B] each
  alignas(1024) uint8_t k[kSlots][kTileBytes];
  alignas(1024) uint8_t q[2][kQBytes];        // [query slot]
  // per-token scales (e4m3) in a ring of their own, twice as deep as the key ring: a key slot is free as soon as its
  // MMAs are done, and the scales of tile i are overwritten by those of tile i + 16, whose copy is issued after the
  // MMAs of tile i + 8 have completed, hence after those of tile i + 4 were issued, which waited for the epilogue of
  // tile i to have read its accumulator and, before that, its scales
  alignas(16) float k_scale[16][kTile];
  float w[2][kHI];
  int32_t ntile[kMaxBatchPs];   // per sequence: tiles, pages and first page of its list, cached length
  int32_t npage[kMaxBatchPs];
  int32_t page0[kMaxBatchPs];
  int32_t ctx[kMaxBatchPs];
  alignas(8) uint64_t k_full[8], k_empty[8], acc_full[4], acc_empty[4], q_full[2], q_empty[2];
  uint32_t tmem_slot;
  int red[kThreadsPs / 32];
  int first_seq, first_tile;
};
static_assert(sizeof(PsSmem<true>) + 1024 <= 227 * 1024 && sizeof(PsSmem<false>) + 1024 <= 227 * 1024, "shared memory");

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
paged_scores_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, IndexArgs p, int flat) {
  using Smem = PsSmem<E4M3>;
  constexpr int kSlots = Smem::kSlots;
  constexpr uint32_t kPageBytes = kPageTok * Smem::kRowBytes;
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
    for (int s = 0; s < kSlots; ++s) {
      tc::mbar_init(smem_u32(&sm.k_full[s]), 1);
      tc::mbar_init(smem_u32(&sm.k_empty[s]), 1);   // the MMAs' commit
    }
    for (int b = 0; b < 4; ++b) {
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.q_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.q_empty[b]), 10);   // once per sequence: the two issuers and the eight epilogue warps
    }
    tc::fence_mbar_init();
  }
  if (warp == 2) {
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

  if (warp < 2) {
    // ================= producers: warp 0 the even tiles of the share, warp 1 the odd ones =================
    const int me = warp;
    bool alive = true;
    for (int base = 0; base < n_tiles && alive; base += 32) {
      // lane l: physical pages of tile base + l
      PsWalker mine = wk;
      for (int s = 0; s < lane; ++s) mine.next(sm.ntile, batch);
      int ph0 = -1, ph1 = -1;
      if (base + lane < n_tiles) {
        int lp0, lp1;
        tile_pages(mine.seq, mine.tile, &lp0, &lp1);
        const int32_t* pt = p.page_table + static_cast<int64_t>(mine.seq) * p.pt_stride;
        ph0 = pt[lp0];
        ph1 = lp1 >= 0 ? pt[lp1] : -1;
      }
      for (int s = 0; s < 32; ++s) wk.next(sm.ntile, batch);   // (walking past the share's end is harmless)
      const int n_here = min(32, n_tiles - base);
      for (int j = me; j < n_here && alive; j += 2) {   // base is even: tile base + j has the parity of j
        const int i = base + j;
        const int f0 = __shfl_sync(0xffffffffu, ph0, j), f1 = __shfl_sync(0xffffffffu, ph1, j);
        bool ok = true;
        if (lane == 0) {
          const int s = i % kSlots;
          ok = tc::mbar_wait(smem_u32(&sm.k_empty[s]), ((i / kSlots) & 1) ^ 1, p.status);
          if (ok) {
            const uint32_t bar = smem_u32(&sm.k_full[s]);
            const uint32_t per_page = kPageBytes + (E4M3 ? kPageTok * 4 : 0);
            tc::mbar_expect_tx(bar, f1 >= 0 ? 2 * per_page : per_page);
            const uint32_t dst = smem_u32(sm.k[s]);
            if constexpr (E4M3) {
              tc::tma_load_2d(dst, &map_k, 0, f0 * kPageTok, bar);
              bulk_load(smem_u32(sm.k_scale[i & 15]), p.k_scale + static_cast<int64_t>(f0) * kPageTok, kPageTok * 4, bar);
              if (f1 >= 0) {
                tc::tma_load_2d(dst + kPageBytes, &map_k, 0, f1 * kPageTok, bar);
                bulk_load(smem_u32(&sm.k_scale[i & 15][kPageTok]), p.k_scale + static_cast<int64_t>(f1) * kPageTok, kPageTok * 4, bar);
              }
            } else {
              // a page = rows 0-63 (or 64-127) of the tile's two 64-dim column blocks
              tc::tma_load_2d(dst, &map_k, 0, f0 * kPageTok, bar);
              tc::tma_load_2d(dst + kAtom, &map_k, 64, f0 * kPageTok, bar);
              if (f1 >= 0) {
                tc::tma_load_2d(dst + kPageTok * 128, &map_k, 0, f1 * kPageTok, bar);
                tc::tma_load_2d(dst + kAtom + kPageTok * 128, &map_k, 64, f1 * kPageTok, bar);
              }
            }
          }
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) alive = false;
      }
    }
  } else if (warp < 4) {
    // ================= MMA issuers: warp 2 the even tiles, warp 3 the odd ones; tile i into accumulator i % 4 =====
    const int me = warp - 2;
    if (lane == 0) {
      constexpr int kSteps = E4M3 ? 12 : 8;
      constexpr uint32_t idesc = E4M3 ? tc::idesc_e4m3_e5m2(kTile, kHI) : tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.k), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      int n_q = 0;
      bool new_seq = true, used = false, ok = true;
      // one arrival per sequence on its query slot: after this thread's last MMA that reads the slot, if there is one
      auto leave_slot = [&](int slot) {
        if (used) tc::umma_commit(smem_u32(&sm.q_empty[slot]));
        else tc::mbar_arrive(smem_u32(&sm.q_empty[slot]));
      };
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (new_seq) {
          if (i > 0) leave_slot((n_q - 1) & 1);
          ++n_q;
          used = false;
          // every sequence's slot is waited for, also one this thread has no tile of: a thread that skipped a phase of
          // the barrier would take an old phase for the one it waits for later (a wait names its phase by parity only)
          ok = tc::mbar_wait(smem_u32(&sm.q_full[(n_q - 1) & 1]), ((n_q - 1) >> 1) & 1, p.status);
          if (!ok) break;
        }
        const int slot = (n_q - 1) & 1;
        new_seq = wk.next(sm.ntile, batch);
        if ((i & 1) != me) continue;
        const int s = i % kSlots, acc = i & 3;
        if (!tc::mbar_wait(smem_u32(&sm.k_full[s]), (i / kSlots) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[acc]), ((i >> 2) & 1) ^ 1, p.status)) {
          ok = false;
          break;
        }
        tc::fence_after_sync();
        const uint32_t d = tmem_base + acc * kHI;
        const uint64_t da = tc::desc_advance(da0, s * Smem::kTileBytes);
        const uint64_t dq = tc::desc_advance(dq0, slot * Smem::kQBytes);
#pragma unroll
        for (int j = 0; j < kSteps; ++j) {
          if constexpr (E4M3)   // plane j / 4, 32-element step j % 4 of the 128-byte rows
            tc::umma_ss_f8(d, tc::desc_advance(da, (j & 3) * 32), tc::desc_advance(dq, (j >> 2) * kAtomQ + (j & 3) * 32), idesc, j != 0);
          else                  // 64-dim column block j / 4, 16-element step j % 4
            tc::umma_ss(d, tc::desc_advance(da, (j >> 2) * kAtom + (j & 3) * 32),
                        tc::desc_advance(dq, (j >> 2) * kAtomQ + (j & 3) * 32), idesc, j != 0);
        }
        tc::umma_commit(smem_u32(&sm.k_empty[s]));
        tc::umma_commit(smem_u32(&sm.acc_full[acc]));
        used = true;
      }
      if (ok) leave_slot((n_q - 1) & 1);
    }
  } else if (warp < 12) {
    // ================= epilogue: warps 4-7 the even tiles, warps 8-11 the odd ones =================
    const int me = (warp >> 2) - 1;
    const int quarter = warp & 3;          // TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;     // token row of the tile
    int n_q = 0;
    bool new_seq = true, ok = true;
    auto leave_slot = [&](int slot) {
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(smem_u32(&sm.q_empty[slot]));
    };
    for (int i = 0; i < n_tiles && ok; ++i) {
      if (new_seq) {
        if (i > 0) leave_slot((n_q - 1) & 1);
        ++n_q;
        // (every sequence's slot is waited for: see the issuers); the head weights were stored before the arrival
        ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.q_full[(n_q - 1) & 1]), ((n_q - 1) >> 1) & 1, p.status));
        if (!ok) break;
      }
      const int slot = (n_q - 1) & 1;
      const int seq = wk.seq, tile = wk.tile;
      new_seq = wk.next(sm.ntile, batch);
      if ((i & 1) != me) continue;
      int lp;
      {
        int lp0, lp1;
        tile_pages(seq, tile, &lp0, &lp1);   // (a page-list entry comes from L2: in flight during the waits below)
        lp = r < kPageTok ? lp0 : lp1;
      }
      const int acc = i & 3;
      const int ctx = sm.ctx[seq];
      const int64_t pos = lp >= 0 ? static_cast<int64_t>(lp) * kPageTok + (r & (kPageTok - 1)) : -1;
      const bool cand = pos >= sh.S && pos <= static_cast<int64_t>(ctx) - 1 - sh.W;
      ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[acc]), (i >> 2) & 1, p.status));
      if (!ok) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + acc * kHI, v);
      tc::tmem_ld_wait();
      const float sc = E4M3 ? sm.k_scale[i & 15][r] : 1.f;   // read before the accumulator is handed back (see k_scale)
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        tc::mbar_arrive(smem_u32(&sm.acc_empty[acc]));
      }
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
      const float score = (a0 + a1) * sc;
      if (flat) {
        if (cand) p.page_scores[static_cast<int64_t>(seq) * p.ps_ld + pos] = score;
      } else if (lp >= 0) {
        p.fine_keys[static_cast<int64_t>(seq) * kMaxSlotsPs + tile * kTile + r] = cand ? score_key(score) : 0u;
      }
    }
    if (ok) leave_slot((n_q - 1) & 1);
  } else {
    // ================= query heads: warps 12-15, one sequence ahead of the tiles =================
    const int qt = tid - (kThreadsPs - kQThreads);   // 0..127
    int n_q = 0;
    bool new_seq = true, ok = true;
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int seq = wk.seq;
      const bool fresh = new_seq;
      new_seq = wk.next(sm.ntile, batch);
      if (!fresh) continue;
      const int slot = n_q & 1;
      ok = tc::mbar_wait(smem_u32(&sm.q_empty[slot]), ((n_q >> 1) & 1) ^ 1, p.status);   // (every thread waits: no hand-over needed)
      if (!ok) break;
      ++n_q;
      if constexpr (E4M3) {
        // 8 threads per head, 16 dims each: three e5m2 planes in the swizzled K-major layout; the head's weight takes
        // the inverse of the head's scale (relu commutes with a positive factor)
        uint8_t* qs = sm.q[slot];
#pragma unroll
        for (int k = 0; k < kHI * 8 / kQThreads; ++k) {
          const int u = qt + k * kQThreads, h = u >> 3, sub = u & 7;
          const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(p.q_idx) +
                                                            (static_cast<int64_t>(seq) * kHI + h) * kDI * 2 + sub * 32);
          const uint4 v0 = src[0], v1 = src[1];
          const uint32_t wv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          float x[16];
          float m = 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            x[2 * j] = __uint_as_float(wv[j] << 16);
            x[2 * j + 1] = __uint_as_float(wv[j] & 0xffff0000u);
            m = fmaxf(m, fmaxf(fabsf(x[2 * j]), fabsf(x[2 * j + 1])));
          }
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
          const int S = e5m2_head_shift(m);
          const float up = __uint_as_float(static_cast<uint32_t>(S + 127) << 23);
#pragma unroll
          for (int j = 0; j < 16; ++j) x[j] *= up;   // exact
          uint4 p1, p2, p3;
          split_e5m2x16(x, p1, p2, p3);
          const int chunk = (sub ^ (h & 7)) << 4;    // rows of all three planes share h & 7 (a plane is 64 rows)
          *reinterpret_cast<uint4*>(qs + 0 * kAtomQ + h * 128 + chunk) = p1;
          *reinterpret_cast<uint4*>(qs + 1 * kAtomQ + h * 128 + chunk) = p2;
          *reinterpret_cast<uint4*>(qs + 2 * kAtomQ + h * 128 + chunk) = p3;
          if (sub == 0)
            sm.w[slot][h] = p.w[static_cast<int64_t>(seq) * kHI + h] * __uint_as_float(static_cast<uint32_t>(127 - S) << 23);
        }
        tc::fence_proxy_async();   // the planes are read by the tensor core
        asm volatile("bar.sync %0, %1;" ::"n"(kQBar), "n"(kQThreads) : "memory");
        if (qt == 0) tc::mbar_arrive(smem_u32(&sm.q_full[slot]));
      } else {
        if (qt < kHI) sm.w[slot][qt] = p.w[static_cast<int64_t>(seq) * kHI + qt];
        asm volatile("bar.sync %0, %1;" ::"n"(kQBar), "n"(kQThreads) : "memory");
        if (qt == 0) {
          tc::mbar_expect_tx(smem_u32(&sm.q_full[slot]), 2 * kAtomQ);
          tc::tma_load_2d(smem_u32(sm.q[slot]), &map_q, 0, seq * kHI, smem_u32(&sm.q_full[slot]));
          tc::tma_load_2d(smem_u32(sm.q[slot]) + kAtomQ, &map_q, 64, seq * kHI, smem_u32(&sm.q_full[slot]));
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 2) tc::tmem_dealloc(tmem_base, kTmemColsPs);
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
  // The key pool belongs to the caller and its size is not part of the call: the map spans the largest row range a
  // page-table entry can address; only boxes of mapped pages are ever requested.
  CUtensorMap map_q, map_k;
  if (!make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kHI) ||
      !(a.key_e4m3 ? make_map_u8_128(&map_k, a.k_idx, 1ull << 31, kPageTok) : make_map_bf16_128(&map_k, a.k_idx, 1ull << 31, kPageTok)))
    return cudaErrorInvalidValue;
  const int64_t max_tiles = flat ? (a.pt_stride + 1) / 2 * a.n_query : static_cast<int64_t>(kMaxPagesPs / 2) * a.n_query;
  int64_t blocks = sm_count > 0 ? sm_count : 148;
  if (blocks > max_tiles) blocks = max_tiles;
  if (blocks < 1) blocks = 1;
  cudaError_t e;
  if (a.key_e4m3) {
    const size_t smem = sizeof(PsSmem<true>) + 1024;
    e = cudaFuncSetAttribute(paged_scores_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = launch_pdl(paged_scores_tc_kernel<true>, dim3(static_cast<unsigned>(blocks)), dim3(kThreadsPs), smem, st, map_q, map_k, a, flat);
  } else {
    const size_t smem = sizeof(PsSmem<false>) + 1024;
    e = cudaFuncSetAttribute(paged_scores_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = launch_pdl(paged_scores_tc_kernel<false>, dim3(static_cast<unsigned>(blocks)), dim3(kThreadsPs), smem, st, map_q, map_k, a, flat);
  }
  ++*n_launch;
  return e;
}

}  // namespace lsa
