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
// Key tiles go from the pool to the tensor cores untouched: a page is one TMA box (64 rows), which lands in the
// 128-byte-swizzled K-major layout the MMA reads.
//   bf16 cache: kind::f16 MMAs against the bf16 query heads (8 x M128 N64 K16 per tile).
//   e4m3 cache: the codes are the A operand of kind::f8f6f4 MMAs as they are.  The bf16 query heads become the B
//     operand as three e5m2 planes: head j is scaled by a power of two 2^S_j that puts its largest element in
//     [2^14, 2^15), then q 2^S = p1 + p2 + p3 with p1 = e5m2(q 2^S), p2 = e5m2(rest), p3 = e5m2(rest of that), each
//     rest exact: a bf16 value has 8 significant bits, a plane takes 3, and an element only loses bits below 2^-23 of
//     its head's largest (below the rounding of the fp32 accumulator).  The three planes accumulate into the same
//     accumulator (12 x M128 N64 K32 per tile), so the tensor core sums them, every product exact, and the epilogue
//     is the same as for bf16 with w_j 2^-S_j in place of w_j (relu commutes with a positive factor).  Nothing is
//     widened and no 16-bit copy of the keys exists anywhere.
//
// Inside a block (12 warps), after the page selection (threads 0-255):
//   warp 0       producer: TMA boxes of the pages into a ring of tiles
//   warps 1-3    one thread of each issues the MMAs of every third tile, alternating between two TMEM accumulators of
//                its own (one thread issues an MMA about every 95 cycles, the pipe needs 48: three issuers keep it
//                busy, and nobody waits for the epilogue of a recent tile)
//   warps 4-7 / 8-11   epilogue of the even / odd tiles: one thread = one token: sum_j w_j relu(acc_j), times the
//                token's scale, as an order-preserving key into the first block's candidate array
// The query heads are fetched before the dependency wait (they are an input of the call, not a product of the
// coarse kernel that precedes this one in the stream).
#include "lsa_internal.h"
#include "lsa_select.cuh"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                  // tokens per tile: two cache pages
constexpr int kPageTok = 64;
constexpr int kThreadsFp = 384;
constexpr int kMaxPagesFp = 64;
constexpr int kMaxSlotsFp = kMaxPagesFp * kPageTok;
constexpr uint32_t kTmemColsFp = 512;       // six accumulators of 64 columns (the allocation is a power of two)
constexpr int kIssuers = 3;                 // MMA-issuing warps 1..3
// Tile i is issued by warp 1 + i % 3 into accumulator (i % 3) + 3 * ((i / 3) % 2): an accumulator belongs to one
// issuer, which alternates between its two.  (A barrier wait names the phase by its parity only: a thread that could
// run two phases ahead of a barrier shared with other issuers would take an old phase for the one it waits for.)
__device__ __forceinline__ int acc_of_tile(int i) { return i % kIssuers + kIssuers * ((i / kIssuers) & 1); }
__device__ __forceinline__ uint32_t acc_use_parity(int i) { return static_cast<uint32_t>(i / (2 * kIssuers)) & 1u; }
constexpr int kSelBar = 1;                  // named barrier of threads 0-255 (the selections)

template <bool E4M3>
struct FpSmem {
  static constexpr int kRowBytes = E4M3 ? kDI : kDI * 2;         // a token's key
  static constexpr int kTileBytes = kTile * kRowBytes;
  // ring slots: a multiple of the number of MMA issuers, so that a slot is always consumed by the same issuer (see
  // acc_of_tile); 144 KB (e4m3) / 96 KB (bf16) of key tiles in flight
  static constexpr int kSlots = E4M3 ? 9 : 3;
  static constexpr int kQBytes = E4M3 ? 3 * kHI * kDI : kHI * kDI * 2;
  // ring of key tiles.  e4m3: [128 rows x 128 B]; bf16: [64-dim half][128 rows x 128 B].  Before the first copy it
  // holds the keys of the page scores (up to kMaxSlotsFp of them).
  alignas(1024) uint8_t k[kSlots][kTileBytes];
  // query heads.  e4m3 cache: three e5m2 planes [plane][64 heads x 128 B]; bf16: [64-dim half][64 heads x 128 B]
  alignas(1024) uint8_t q[kQBytes];
  float k_scale[E4M3 ? kMaxPagesFp / 2 : 1][kTile];   // per-token scales of the block's tiles (e4m3); a thread reads what it wrote
  float w[kHI];
  uint32_t keys[kMaxSlotsFp];   // candidate keys of the whole cluster (used in the first block only)
  int32_t pages[kMaxPagesFp];   // kept pages, ascending
  int32_t phys[kMaxPagesFp];    // their places in the pool
  SelectScratch sel;
  alignas(8) uint64_t k_full[9], k_empty[9], acc_full[2 * kIssuers], acc_empty[2 * kIssuers], q_full;
  uint32_t tmem_slot;
};
static_assert(sizeof(FpSmem<true>) + 1024 <= 227 * 1024 && sizeof(FpSmem<false>) + 1024 <= 227 * 1024, "shared memory");
static_assert(FpSmem<true>::kSlots * FpSmem<true>::kTileBytes >= kMaxSlotsFp * 4, "page keys fit the ring");
static_assert(FpSmem<true>::kSlots % kIssuers == 0 && FpSmem<false>::kSlots % kIssuers == 0, "a ring slot has one consumer");

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
fine_paged_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, IndexArgs p) {
  using Smem = FpSmem<E4M3>;
  constexpr int kSlots = Smem::kSlots;
  constexpr int kAtom = kTile * 128;        // 128 rows x 128 B
  constexpr int kAtomQ = kHI * 128;
  extern __shared__ uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.y;
  const uint32_t rank = cluster_rank(), n_rank = cluster_size();
  // The cluster barrier has no time limit: every path below reaches both of its phases, also after a failed wait.
  cluster_arrive();   // phase 1: "this block runs" (its shared memory may be written from now on)
  const bool live = !tc::status_raised(p.status);

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) {
      tc::mbar_init(smem_u32(&sm.k_full[s]), 1);
      tc::mbar_init(smem_u32(&sm.k_empty[s]), 1);   // the MMAs' commit
    }
    for (int b = 0; b < 2 * kIssuers; ++b) {
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
    }
    tc::mbar_init(smem_u32(&sm.q_full), 1);
    tc::fence_mbar_init();
    if (!E4M3 && live) {
      tc::mbar_expect_tx(smem_u32(&sm.q_full), 2 * kAtomQ);
      tc::tma_load_2d(smem_u32(sm.q), &map_q, 0, qi * kHI, smem_u32(&sm.q_full));
      tc::tma_load_2d(smem_u32(sm.q) + kAtomQ, &map_q, 64, qi * kHI, smem_u32(&sm.q_full));
    }
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsFp);
    tc::tmem_relinquish();
  }
  if constexpr (E4M3) {
    // query heads -> three e5m2 planes in the swizzled K-major layout; head weights take the inverse of the head's scale
    for (int u = tid; u < kHI * 8; u += kThreadsFp) {   // 8 threads per head, 16 dims each (a warp never straddles a head group)
      const int h = u >> 3, sub = u & 7;
      const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(p.q_idx) +
                                                        (static_cast<int64_t>(qi) * kHI + h) * kDI * 2 + sub * 32);
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
      *reinterpret_cast<uint4*>(sm.q + 0 * kAtomQ + h * 128 + chunk) = p1;
      *reinterpret_cast<uint4*>(sm.q + 1 * kAtomQ + h * 128 + chunk) = p2;
      *reinterpret_cast<uint4*>(sm.q + 2 * kAtomQ + h * 128 + chunk) = p3;
      if (sub == 0) sm.w[h] = p.w[static_cast<int64_t>(qi) * kHI + h] * __uint_as_float(static_cast<uint32_t>(127 - S) << 23);
    }
    tc::fence_proxy_async();   // the planes are read by the tensor core
  } else {
    if (tid < kHI) sm.w[tid] = p.w[static_cast<int64_t>(qi) * kHI + tid];
  }
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
          uint32_t* pk = reinterpret_cast<uint32_t*>(sm.k);
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
          tc::fence_proxy_async();   // the ring is handed to the TMA copies
        } else {
          nP = block_select_topk<kSelBar, true>([&](int i) { return score_key(ps[i]); }, [&](int i) { return p0 + i; }, nE, p.M,
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
    if (tid == 0) sm.sel.n_valid = static_cast<uint32_t>(nP);   // for the other warps of the block
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
      constexpr uint32_t kPageBytes = kPageTok * Smem::kRowBytes;
      for (int i = 0; i < n_tiles; ++i) {
        const int tl = tile0 + i;
        const int f0 = sm.phys[2 * tl];
        const int f1 = 2 * tl + 1 < nP ? sm.phys[2 * tl + 1] : -1;
        const int s = i % kSlots;
        if (!tc::mbar_wait(smem_u32(&sm.k_empty[s]), ((i / kSlots) & 1) ^ 1, p.status)) break;
        const uint32_t bar = smem_u32(&sm.k_full[s]);
        tc::mbar_expect_tx(bar, f1 >= 0 ? 2 * kPageBytes : kPageBytes);
        const uint32_t dst = smem_u32(sm.k[s]);
        if constexpr (E4M3) {
          tc::tma_load_2d(dst, &map_k, 0, f0 * kPageTok, bar);
          if (f1 >= 0) tc::tma_load_2d(dst + kPageBytes, &map_k, 0, f1 * kPageTok, bar);
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
  } else if (warp <= kIssuers) {
    // ================= MMA issuers: warps 1-3 take every third tile each, alternating between two accumulators of
    // their own, so that nobody waits for the epilogue of a recent tile.  One thread issues an MMA about every 95
    // cycles here and the pipe needs 48 for one (both operands from shared memory): three issuers keep it busy ====
    const int b = warp - 1;
    if (lane == 0 && n_tiles > b) {
      constexpr int kSteps = E4M3 ? 12 : 8;
      constexpr uint32_t idesc = E4M3 ? tc::idesc_e4m3_e5m2(kTile, kHI) : tc::idesc_bf16(kTile, kHI, 0, 0);
      const uint64_t da0 = tc::smem_desc_sw128(smem_u32(sm.k), 16, 1024);
      const uint64_t dq0 = tc::smem_desc_sw128(smem_u32(sm.q), 16, 1024);
      uint32_t a_off[kSteps];
      uint64_t dq[kSteps];
#pragma unroll
      for (int j = 0; j < kSteps; ++j) {
        if constexpr (E4M3) {   // plane j / 4, 32-element step j % 4 of the 128-byte rows
          a_off[j] = (j & 3) * 32;
          dq[j] = tc::desc_advance(dq0, (j >> 2) * kAtomQ + (j & 3) * 32);
        } else {                // 64-dim column block j / 4, 16-element step j % 4
          a_off[j] = (j >> 2) * kAtom + (j & 3) * 32;
          dq[j] = tc::desc_advance(dq0, (j >> 2) * kAtomQ + (j & 3) * 32);
        }
      }
      bool ok = E4M3 ? true : tc::mbar_wait(smem_u32(&sm.q_full), 0, p.status);
      for (int i = b; i < n_tiles && ok; i += kIssuers) {
        const int s = i % kSlots;
        const int acc = acc_of_tile(i);
        if (!tc::mbar_wait(smem_u32(&sm.k_full[s]), (i / kSlots) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[acc]), acc_use_parity(i) ^ 1u, p.status))
          break;
        tc::fence_after_sync();
        const uint32_t d = tmem_base + acc * kHI;
        const uint64_t da = tc::desc_advance(da0, s * Smem::kTileBytes);
#pragma unroll
        for (int j = 0; j < kSteps; ++j) {
          if constexpr (E4M3) tc::umma_ss_f8(d, tc::desc_advance(da, a_off[j]), dq[j], idesc, j != 0);
          else tc::umma_ss(d, tc::desc_advance(da, a_off[j]), dq[j], idesc, j != 0);
        }
        tc::umma_commit(smem_u32(&sm.k_empty[s]));
        tc::umma_commit(smem_u32(&sm.acc_full[acc]));
      }
    }
  } else if (warp >= 4) {
    // ================= epilogue: warps 4-7 the even tiles, warps 8-11 the odd ones =================
    const int b = (warp >> 2) - 1;
    const int quarter = warp & 3;          // TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;     // token row of the tile
    const uint32_t keys0 = smem_of_rank(smem_u32(sm.keys), 0);
    if constexpr (E4M3) {
      // the scales of this thread's tokens, straight from the pool (an issued TMA or bulk copy costs its thread some
      // 200 cycles, so the producer issues nothing but the key boxes); the loads of all tiles are in flight together
      for (int i0 = b; i0 < n_tiles; i0 += 16) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {   // eight loads in flight
          const int i = i0 + 2 * u;
          const int c = (tile0 + i) * kTile + r;
          v[u] = (i < n_tiles && c < n_slots) ? p.k_scale[static_cast<int64_t>(sm.phys[c >> 6]) * kPageTok + (c & (kPageTok - 1))] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (i0 + 2 * u < n_tiles) sm.k_scale[i0 + 2 * u][r] = v[u];
      }
    }
    for (int i = b; i < n_tiles; i += 2) {
      const int acc = acc_of_tile(i);
      const int c = (tile0 + i) * kTile + r;   // candidate slot
      int64_t pos = -1;
      if (c < n_slots) pos = static_cast<int64_t>(sm.pages[c >> 6]) * kPageTok + (c & (kPageTok - 1));
      const bool cand = pos >= lo && pos <= hi;
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[acc]), acc_use_parity(i), p.status))) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + acc * kHI, v);
      tc::tmem_ld_wait();
      const float sc = E4M3 ? sm.k_scale[i][r] : 1.f;
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        tc::mbar_arrive(smem_u32(&sm.acc_empty[acc]));
      }
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
  // The key pool belongs to the caller and its size is not part of the call: the map spans the largest row range a
  // page-table entry can address; only boxes of mapped pages are ever requested.
  CUtensorMap map_q, map_k;
  if (!make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kHI) ||
      !(a.key_e4m3 ? make_map_u8_128(&map_k, a.k_idx, 1ull << 31, kPageTok) : make_map_bf16_128(&map_k, a.k_idx, 1ull << 31, kPageTok)))
    return cudaErrorInvalidValue;
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
    e = cudaLaunchKernelEx(&cfg, fine_paged_tc_kernel<true>, map_q, map_k, a);
  } else {
    cfg.dynamicSmemBytes = sizeof(FpSmem<false>) + 1024;
    e = cudaFuncSetAttribute(fine_paged_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(cfg.dynamicSmemBytes));
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, fine_paged_tc_kernel<false>, map_q, map_k, a);
  }
  ++*n_launch;
  return e;
}

}  // namespace lsa
