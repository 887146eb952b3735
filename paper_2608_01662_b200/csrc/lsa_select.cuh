// Block-wide exact top-k by radix select, with ordered compaction.
//
// Items i = 0..n-1 carry a 32-bit key (larger = better, 0 = absent) and appear in ascending id
// order.  The k items that are largest under (key descending, i ascending) are written in
// ascending i.  Four 8-bit histogram passes find the k-th largest key T; everything above T is
// taken, and of the items equal to T the first (k - #above) in index order.  Three block barriers per pass.
//
// The code runs once per block, and what it costs there is to a large part the fetch of its instructions.  Measured
// inside the decode kernels (4096 keys, k = 2048; cycles from a cold / a warm instruction cache): this version
// 18.3 k / 14.9 k; a version that skips the bits all keys share, ranks a small threshold bin directly and unrolls
// the compaction 16 rows deep 29.9 k / 13.1 k (its code is twice as large); the same with every loop rolled
// 20.8 k / 19.5 k.  So the plain version stays.
#pragma once

#include "lsa_common.cuh"

namespace lsa {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;

struct SelectScratch {
  uint32_t hist[kSelWarps][256];
  uint32_t warp_gt[kSelWarps];
  uint32_t warp_eq[kSelWarps];
  uint32_t prefix;
  uint32_t remaining;
  uint32_t n_valid;
};

// Barrier of the 256 selecting threads: the whole block (BAR = 0), or threads 0-255 of a larger block on the named
// barrier BAR.
template <int BAR>
__device__ __forceinline__ void select_sync() {
  if constexpr (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(kSelThreads) : "memory");
}
// KeyF: uint32_t operator()(int i).   EmitF: void operator()(int r, int i): item i is the r-th of the selection
// (ascending i).   AbsentF: void operator()(int r): there is no r-th item (r in [written, k)).
// Every thread of the 256-thread block must call this (BAR != 0: threads 0-255 of a larger block, all of them).
// Returns the number of items selected (min(k, #present)).
// Key of item i of [0, n), 0 beyond.  UNCOND: the functor is called for every i (on the last item beyond the range),
// so that the global-memory loads inside it are not control-dependent and the loads of one step are issued together
// (a functor that reads a long row from L2 runs 2.5 x faster that way; for keys in shared memory it does not pay).
template <bool UNCOND, class KeyF>
__device__ __forceinline__ uint32_t select_key(KeyF& key, int i, int n) {
  if constexpr (UNCOND) {
    const uint32_t v = key(min(i, n - 1));
    return i < n ? v : 0u;
  } else {
    return i < n ? key(i) : 0u;
  }
}

template <int BAR = 0, bool UNCOND = false, class KeyF, class EmitF, class AbsentF>
__device__ int block_select_topk_emit(KeyF key, EmitF emit, AbsentF absent, int n, int k, SelectScratch& sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- radix select: four 8-bit passes from the top byte down.  A pass counts the digits of the keys that still
  // match the prefix into per-warp histograms (zero between passes: every thread clears the bins it has just summed);
  // then thread t sums bin 255 - t over the warps, the block scans those sums from the top bin down (warp shuffles
  // plus one exchange of warp totals), and the thread whose bin holds the k-th key publishes the new prefix.  The
  // first pass also yields the number of keys present (its grand total): with k or fewer, everything is taken.
  uint32_t T = 0;      // take keys > T ...
  int need_eq = 0;     // ... and the first need_eq keys == T
  for (int i = tid; i < kSelWarps * 256; i += kSelThreads) (&sc.hist[0][0])[i] = 0;
  if (tid == 0) sc.n_valid = 0;
  select_sync<BAR>();
  int n_valid = 0;
  {
    uint32_t prefix = 0, mask = 0;
    uint32_t remaining = static_cast<uint32_t>(k > 0 ? k : 0);
    bool take_all = false;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      // four keys per thread and step: when the keys come from global memory the loads are in flight together
      for (int i0 = tid; i0 < n; i0 += 4 * kSelThreads) {
        uint32_t kk[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kSelThreads;
          kk[u] = select_key<UNCOND>(key, i, n);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (kk[u] != 0u && (kk[u] & mask) == prefix) atomicAdd(&sc.hist[warp][(kk[u] >> shift) & 255u], 1u);
      }
      select_sync<BAR>();
      // bin 255 - tid: its count over all warps, cleared for the next pass
      const int bin = 255 - tid;
      uint32_t cnt = 0;
#pragma unroll
      for (int w = 0; w < kSelWarps; ++w) {
        cnt += sc.hist[w][bin];
        sc.hist[w][bin] = 0;
      }
      uint32_t incl = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
      }
      if (lane == 31) sc.warp_gt[warp] = incl;   // this warp's 32 bins
      select_sync<BAR>();
      uint32_t before = 0, total = 0;
#pragma unroll
      for (int w = 0; w < kSelWarps; ++w) {
        const uint32_t v = sc.warp_gt[w];
        before += w < warp ? v : 0u;
        total += v;
      }
      incl += before;
      const uint32_t excl = incl - cnt;
      if (shift == 24) {
        n_valid = static_cast<int>(total);
        take_all = n_valid <= k || k <= 0;
      }
      if (!take_all && excl < remaining && remaining <= incl) {   // exactly one thread
        sc.prefix = prefix | (static_cast<uint32_t>(bin) << shift);
        sc.remaining = remaining - excl;
      }
      select_sync<BAR>();
      if (take_all) break;   // uniform: every thread computed the same total
      prefix = sc.prefix;
      remaining = sc.remaining;
      mask |= 255u << shift;
    }
    if (!take_all) {
      T = prefix;
      need_eq = static_cast<int>(remaining);
    }
  }
  if (k <= 0 || n_valid == 0) {
    for (int i = tid; i < k; i += kSelThreads) absent(i);
    select_sync<BAR>();
    return 0;
  }

  // ---- ordered compaction: warp w owns the contiguous index range [w*per, (w+1)*per)
  const int per = ((n + kSelWarps - 1) / kSelWarps + 31) & ~31;
  const int begin = warp * per, end = min(n, begin + per);
  uint32_t gt = 0, eq = 0;
  for (int i0 = begin + lane; i0 < end; i0 += 4 * 32) {
    uint32_t kk[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u;
      kk[u] = select_key<UNCOND>(key, i, end);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      gt += kk[u] > T;
      eq += (kk[u] == T) & (kk[u] != 0u);
    }
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  eq = __reduce_add_sync(0xffffffffu, eq);
  if (lane == 0) {
    sc.warp_gt[warp] = gt;
    sc.warp_eq[warp] = eq;
  }
  select_sync<BAR>();
  int gt_before = 0, eq_before = 0;
  for (int w = 0; w < warp; ++w) {
    gt_before += static_cast<int>(sc.warp_gt[w]);
    eq_before += static_cast<int>(sc.warp_eq[w]);
  }
  int out_run = gt_before + min(eq_before, need_eq);
  int eq_run = eq_before;
  const uint32_t lt_mask = (1u << lane) - 1u;
  // four rows of 32 keys per step: their loads and the ballots of the threshold ties do not wait for one another
#pragma unroll 1
  for (int base = begin; base < end; base += 4 * 32) {
    uint32_t kk[4], eq_mask[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = base + 32 * u + lane;
      kk[u] = select_key<UNCOND>(key, i, end);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) eq_mask[u] = __ballot_sync(0xffffffffu, (kk[u] == T) && (kk[u] != 0u));
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool is_eq = (kk[u] == T) && (kk[u] != 0u);
      const bool sel = kk[u] > T || (is_eq && eq_run + __popc(eq_mask[u] & lt_mask) < need_eq);
      const uint32_t sel_mask = __ballot_sync(0xffffffffu, sel);
      if (sel) emit(out_run + __popc(sel_mask & lt_mask), base + 32 * u + lane);
      out_run += __popc(sel_mask);
      eq_run += __popc(eq_mask[u]);
    }
  }
  const int written = min(k, n_valid);
  for (int i = written + tid; i < k; i += kSelThreads) absent(i);
  select_sync<BAR>();
  return written;
}

// The common form: out[r] = id(i) for the selected items in ascending i, out[written..k) = -1.
// IdF: int operator()(int i).
template <int BAR = 0, bool UNCOND = false, class KeyF, class IdF>
__device__ int block_select_topk(KeyF key, IdF id, int n, int k, int* out, SelectScratch& sc) {
  return block_select_topk_emit<BAR, UNCOND>(key, [&](int r, int i) { out[r] = id(i); }, [&](int r) { out[r] = -1; }, n, k, sc);
}
}  // namespace lsa
