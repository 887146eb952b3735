// a1 for paged (decode) caches on the 5th-generation tensor cores, 64-head / 128-dim indexer.
//
// Decode has one query per sequence, so the large operand is the cache of sub-block mean keys (Sec. 3.3): the stage is
// an HBM read of all of it with a thin GEMM on top.  Sequences differ in length by an order of magnitude, so the work
// is cut by tiles, not by sequences: the 128-row mean-key tiles of all sequences form one list, and each of the
// 2 x SM-count resident blocks takes an equal contiguous share of it (every block derives the same partition from the
// cached lengths; nothing is scheduled dynamically).  Inside a block:
//
//   warps 0, 6-8  producers: for each tile, look up the physical page of each of its logical pages and issue one TMA box
//               per page and 64-dim half (the sub-blocks of a page are consecutive rows of the mean cache) into a
//               two-deep ring.  A box is 1 KB and a TMA instruction costs its issuing warp some eighty cycles, so the
//               32 boxes of a tile are spread over four warps.  When the block's share crosses into the next sequence,
//               warp 0 fetches that sequence's query heads (TMA) and head weights into the other of two query slots
//   warp 1      one thread issues 8 x tcgen05.mma (M128 N64 K16) per tile into one of two TMEM accumulators
//   warps 2-5   epilogue: one thread = one sub-block row: sum_j w_j relu(acc_j), then the sum over the page's
//               sub-blocks (Eq. 9) with warp shuffles, page score to global
#include "lsa_internal.h"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTile = 128;                  // sub-block rows per tile
constexpr int kAtomA = kTile * 128;         // one 64-dim column block of a tile
constexpr int kAtomQ = kHI * 128;
constexpr int kStages = 2;                  // two blocks share an SM: four tiles (128 KB) in flight per SM
constexpr int kThreadsCp = 288;             // warps 0, 6, 7, 8: producers; 1: MMA; 2-5: epilogue
constexpr int kProducerWarps = 4;
constexpr int kMaxBatchCp = 2048;           // cached lengths kept in shared memory
constexpr uint32_t kTmemColsCp = 128;       // two accumulators of 64 columns

struct CoarsePagedTcSmem {
  alignas(1024) uint8_t a[kStages][2][kAtomA];
  alignas(1024) uint8_t q[2][2][kAtomQ];    // [query slot][64-dim half]
  float w[2][kHI];
  int32_t ctx[kMaxBatchCp];
  alignas(8) uint64_t full[kStages], empty[kStages], acc_full[2], acc_empty[2], q_full[2], q_empty[2];
  uint32_t tmem_slot;
  int red[kThreadsCp / 32];
  int first_seq, first_tile;
};

struct Shape {
  int S, W, M, B, p_shift, spp_shift;
};

// 128-row tiles of mean keys the coarse stage reads for a sequence of `ctx` cached tokens (0: the stage is skipped,
// because no more than M pages are eligible)
__device__ __forceinline__ int tiles_of(int ctx, const Shape& sh) {
  const int hi = ctx - 1 - sh.W;
  if (hi < sh.S || (hi >> sh.p_shift) - (sh.S >> sh.p_shift) + 1 <= sh.M) return 0;
  return ((hi >> sh.p_shift) >> (7 - sh.spp_shift)) + 1;
}

// Walks a block's share of the tile list: (seq, tile) of the current tile, moving on to the next sequence that has tiles.
struct Walker {
  int seq, tile, n_in_seq;
  __device__ __forceinline__ void start(const int32_t* ctx, const Shape& sh, int s, int tl) {
    seq = s;
    tile = tl;
    n_in_seq = tiles_of(ctx[s], sh);
  }
  // returns true when the next tile belongs to another sequence
  __device__ __forceinline__ bool next(const int32_t* ctx, const Shape& sh, int batch) {
    if (++tile < n_in_seq) return false;
    tile = 0;
    do {
      ++seq;
      n_in_seq = seq < batch ? tiles_of(ctx[seq], sh) : 1;   // past the end: only reached after a block's last tile
    } while (n_in_seq == 0);
    return true;
  }
};

__global__ void __launch_bounds__(kThreadsCp, 2)
coarse_score_paged_tc_kernel(const __grid_constant__ CUtensorMap map_km, const __grid_constant__ CUtensorMap map_q, IndexArgs p) {
  extern __shared__ uint8_t smem_raw[];
  CoarsePagedTcSmem& sm = *reinterpret_cast<CoarsePagedTcSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int batch = p.n_query;
  Shape sh;
  sh.S = p.S; sh.W = p.W; sh.M = p.M; sh.B = p.B;
  sh.p_shift = 31 - __clz(p.P);
  const int spp = p.P / p.B;                       // sub-blocks per page: 8, 16 or 32
  sh.spp_shift = 31 - __clz(spp);
  if (tc::status_raised(p.status)) return;
  pdl_wait();                 // the cached lengths may come from the previous kernel of the stream (lsa_append)
  pdl_launch_dependents();

  // ---- this block's share of the tile list
  int my_tiles = 0;
  for (int s = tid; s < batch; s += kThreadsCp) {
    const int c = p.ctx_len[s];
    sm.ctx[s] = c;
    my_tiles += tiles_of(c, sh);
  }
  my_tiles = __reduce_add_sync(0xffffffffu, my_tiles);
  if (lane == 0) sm.red[warp] = my_tiles;
  __syncthreads();
  int total = 0;
  for (int i = 0; i < kThreadsCp / 32; ++i) total += sm.red[i];
  const int g0 = static_cast<int>(static_cast<int64_t>(total) * blockIdx.x / gridDim.x);
  const int g1 = static_cast<int>(static_cast<int64_t>(total) * (blockIdx.x + 1) / gridDim.x);
  const int n_tiles = g1 - g0;
  if (n_tiles <= 0) return;
  if (warp == 0) {
    // sequence and tile that hold list position g0: a warp-wide scan, 32 sequences per round
    int base = 0, found_seq = -1, found_tile = 0;
    for (int s0 = 0; s0 < batch && found_seq < 0; s0 += 32) {
      const int n = s0 + lane < batch ? tiles_of(sm.ctx[s0 + lane], sh) : 0;
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
    for (int s = 0; s < kStages; ++s) {
      tc::mbar_init(smem_u32(&sm.full[s]), 1);
      tc::mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), 4);
      tc::mbar_init(smem_u32(&sm.q_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.q_empty[b]), 5);   // the MMA thread's commit and the four epilogue warps
    }
    tc::fence_mbar_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsCp);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;
  Walker wk;
  wk.start(sm.ctx, sh, sm.first_seq, sm.first_tile);

  const int pw = warp == 0 ? 0 : warp - 5;   // producer number of warps 0, 6, 7, 8
  if (warp == 0 || warp >= 6) {
    // ================= producers =================
    const int pages_per_tile = kTile >> sh.spp_shift;    // 16, 8 or 4
    const int n_loads = pages_per_tile * 2;              // one box per page and 64-dim half
    const int per_warp = n_loads / kProducerWarps;       // 8, 4 or 2 boxes per producer warp
    const int box = pw * per_warp + lane;                // the box this lane issues (lanes below per_warp)
    const bool issues = lane < per_warp;
    const int box_bytes = spp * 128;
    auto first_row = [&](int seq, int tile) -> int {     // physical row of the box this lane fetches
      const int n_sub = (sm.ctx[seq] + sh.B - 1) / sh.B;
      const int sub0 = tile * kTile + ((box >> 1) << sh.spp_shift);
      // pages past the cached length are never eligible: any mapped rows will do, the epilogue drops them
      return (issues && sub0 < n_sub) ? p.page_table[seq * p.pt_stride + (sub0 >> sh.spp_shift)] << sh.spp_shift : 0;
    };
    int n_q = 0;
    bool new_seq = true;
    int row_next = first_row(wk.seq, wk.tile);
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kStages;
      const int row = row_next;
      const int seq = wk.seq;
      const bool was_new = new_seq;
      new_seq = wk.next(sm.ctx, sh, batch);
      if (i + 1 < n_tiles) row_next = first_row(wk.seq, wk.tile);   // look-ups of the next tile: off the critical path
      bool ok = true;
      if (was_new && pw == 0) {
        // query heads and head weights of this sequence into slot n_q & 1
        const int slot = n_q & 1;
        if (lane == 0) ok = tc::mbar_wait(smem_u32(&sm.q_empty[slot]), ((n_q >> 1) & 1) ^ 1, p.status);
        if (!__shfl_sync(0xffffffffu, ok, 0)) break;
        sm.w[slot][lane] = p.w[static_cast<int64_t>(seq) * kHI + lane];
        sm.w[slot][lane + 32] = p.w[static_cast<int64_t>(seq) * kHI + lane + 32];
        __syncwarp();
        if (lane == 0) {
          tc::mbar_expect_tx(smem_u32(&sm.q_full[slot]), 2 * kAtomQ);
          tc::tma_load_2d(smem_u32(sm.q[slot][0]), &map_q, 0, seq * kHI, smem_u32(&sm.q_full[slot]));
          tc::tma_load_2d(smem_u32(sm.q[slot][1]), &map_q, 64, seq * kHI, smem_u32(&sm.q_full[slot]));
        }
        ++n_q;
      }
      if (lane == 0) {
        ok = tc::mbar_wait(smem_u32(&sm.empty[s]), ((i / kStages) & 1) ^ 1, p.status);
        // one arrival per tile, by producer 0; bytes the other producers' boxes complete before it are counted all the same
        if (ok && pw == 0) tc::mbar_expect_tx(smem_u32(&sm.full[s]), 2 * kAtomA);
      }
      if (!__shfl_sync(0xffffffffu, ok, 0)) break;
      if (issues)
        tc::tma_load_2d(smem_u32(sm.a[s][box & 1]) + (box >> 1) * box_bytes, &map_km, (box & 1) * 64, row, smem_u32(&sm.full[s]));
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
        const int s = i % kStages, b = i & 1;
        if (new_seq) {
          if (!tc::mbar_wait(smem_u32(&sm.q_full[n_q & 1]), (n_q >> 1) & 1, p.status)) break;
          ++n_q;
        }
        const int slot = (n_q - 1) & 1;
        new_seq = wk.next(sm.ctx, sh, batch);
        if (!tc::mbar_wait(smem_u32(&sm.full[s]), (i / kStages) & 1, p.status) ||
            !tc::mbar_wait(smem_u32(&sm.acc_empty[b]), ((i >> 1) & 1) ^ 1, p.status))
          break;
        tc::fence_after_sync();
        const uint32_t d = tmem_base + b * kHI;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // 16-dim step: column block ks/4, 32-byte slice ks%4
          tc::umma_ss(d, tc::desc_advance(da0, s * 2 * kAtomA + (ks >> 2) * kAtomA + (ks & 3) * 32),
                      tc::desc_advance(dq0, slot * 2 * kAtomQ + (ks >> 2) * kAtomQ + (ks & 3) * 32), idesc, ks != 0);
        tc::umma_commit(smem_u32(&sm.empty[s]));
        tc::umma_commit(smem_u32(&sm.acc_full[b]));
        if (new_seq || i + 1 == n_tiles) tc::umma_commit(smem_u32(&sm.q_empty[slot]));   // last tile of its sequence here
      }
    }
  } else if (warp < 6) {
    // ================= epilogue warps =================
    const int quarter = warp & 3;          // warps 2-5 own TMEM lanes 32*quarter .. +31
    const int r = 32 * quarter + lane;     // sub-block row of the tile
    int n_q = 0;
    bool new_seq = true;
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i & 1;
      if (new_seq) {
        // the head weights of the slot were stored before the arrival on q_full
        if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.q_full[n_q & 1]), (n_q >> 1) & 1, p.status))) break;
        ++n_q;
      }
      const int slot = (n_q - 1) & 1;
      const int seq = wk.seq, tile = wk.tile;
      new_seq = wk.next(sm.ctx, sh, batch);
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[b]), (i >> 1) & 1, p.status))) break;
      tc::fence_after_sync();
      uint32_t v[64];
      tc::tmem_ld64(tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + b * kHI, v);
      tc::tmem_ld_wait();
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
      const int ctx = sm.ctx[seq];
      const int n_sub = (ctx + sh.B - 1) / sh.B;
      const int hi = ctx - 1 - sh.W;
      const int sub = tile * kTile + r;
      float sc = sub < n_sub ? a0 + a1 : 0.f;   // rows past the cache hold whatever the pool had there
      for (int d = 1; d < spp; d <<= 1) sc += __shfl_xor_sync(0xffffffffu, sc, d);
      if ((lane & (spp - 1)) == 0) {
        const int page = sub >> sh.spp_shift;
        if ((page << sh.p_shift) <= hi) p.page_scores[static_cast<int64_t>(seq) * p.ps_ld + page] = sc;
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemColsCp);
}

int sm_count_of_current_device() {
  static int counts[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (counts[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    counts[dev] = n;
  }
  return counts[dev];
}

}  // namespace

bool coarse_paged_tc_supported(const IndexArgs& a) {
  return a.paged && a.HI == kHI && a.DI == kDI && a.n_query <= kMaxBatchCp && (a.P & (a.P - 1)) == 0 &&
         (reinterpret_cast<uintptr_t>(a.kmean) & 15u) == 0 && (reinterpret_cast<uintptr_t>(a.q_idx) & 15u) == 0 &&
         tma_available();
}

cudaError_t launch_coarse_paged_tc(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  CUtensorMap map_km, map_q;
  // The pool of mean keys belongs to the caller and its size is not part of the call: the map spans the largest
  // row range a page table entry can address; only boxes of mapped pages are ever requested.
  const int spp = a.P / a.B;
  if (!make_map_bf16_128(&map_km, a.kmean, 1ull << 31, static_cast<uint32_t>(spp)) ||
      !make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kHI))
    return cudaErrorInvalidValue;
  const size_t smem = sizeof(CoarsePagedTcSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(coarse_score_paged_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int64_t n_sub_max = (a.pt_stride * a.P + a.B - 1) / a.B;
  const int64_t max_tiles = (n_sub_max + kTile - 1) / kTile * a.n_query;   // upper bound on the tile list
  int64_t blocks = 2 * sm_count_of_current_device();
  if (blocks > max_tiles) blocks = max_tiles;
  if (blocks < 1) blocks = 1;
  e = launch_pdl(coarse_score_paged_tc_kernel, dim3(static_cast<unsigned>(blocks)), dim3(kThreadsCp), smem, st, map_km, map_q, a);
  ++*n_launch;
  return e;
}

}  // namespace lsa
