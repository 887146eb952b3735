// Exact top-k of one long row by a thread-block cluster: the same selection as block_select_topk (lsa_select.cuh:
// largest keys first, ties by position, output in ascending position), with the row cut into one contiguous piece
// per block of the cluster.
//
// Each of the four 8-bit radix passes: every block counts the digits of its piece (per-warp histograms in its own
// shared memory), adds its 256 bin totals to the histogram in the first block's shared memory (remote atomics), the
// first block scans the bins and publishes the new prefix, everybody reads it back.  Two cluster barriers per pass.
// The compaction needs one more exchange: each block's counts of keys above and equal to the threshold, from which a
// block knows where its part of the output starts and how many of the threshold's ties are its own to take.
//
// For rows of 10^4 .. 10^6 scores with few rows in flight (the flat indexer in decode): one block per row re-reads
// the whole row seven times by itself; here the passes run on eight SMs at once.
#pragma once

#include "lsa_select.cuh"

namespace lsa {

constexpr int kClusterSel = 8;   // blocks per row (the portable cluster size)

struct ClusterSelScratch {
  uint32_t hist[kSelWarps][256];      // this block's per-warp histograms
  uint32_t total[256];                // first block: the cluster's histogram of the current pass
  uint32_t cnt[kClusterSel][2];       // first block: keys above / equal to the threshold, per block
  uint32_t warp_gt[kSelWarps], warp_eq[kSelWarps];
  uint32_t prefix, remaining, n_valid, take_all;   // first block: published after each scan
};

namespace cluster_sel {
__device__ __forceinline__ uint32_t rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void sync() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t at_rank0(const void* p) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(0));
  return r;
}
__device__ __forceinline__ void add_remote(uint32_t addr, uint32_t v) {
  asm volatile("red.relaxed.cluster.shared::cluster.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void store_remote(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t load_remote(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
}  // namespace cluster_sel

// KeyF: uint32_t operator()(int i) (0 = absent).   IdF: int operator()(int i).
// Every thread of every block of the cluster (kClusterSel blocks of kSelThreads threads along x) must call this with
// the same arguments.  out[0 .. written) = ids of the selection in ascending i, out[written .. k) = -1; returns written.
template <class KeyF, class IdF>
__device__ int cluster_select_topk(KeyF key, IdF id, int n, int k, int* out, ClusterSelScratch& sc) {
  namespace cs = cluster_sel;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t me = cs::rank();
  // this block's piece of the row
  const int chunk = ((n + kClusterSel - 1) / kClusterSel + 255) & ~255;
  const int b0 = min(n, static_cast<int>(me) * chunk), b1 = min(n, b0 + chunk);

  for (int i = tid; i < kSelWarps * 256; i += kSelThreads) (&sc.hist[0][0])[i] = 0;
  if (me == 0) {
    sc.total[tid] = 0;
    if (tid == 0) sc.take_all = 0;
  }
  __syncthreads();
  cs::sync();   // every block of the cluster runs and the first block's histogram is clear

  const uint32_t total0 = cs::at_rank0(sc.total), pub0 = cs::at_rank0(&sc.prefix);
  uint32_t T = 0;      // take keys > T ...
  int need_eq = 0;     // ... and the first need_eq keys == T
  int n_valid = 0;
  bool take_all = false;
  {
    uint32_t prefix = 0, mask = 0;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i0 = b0 + tid; i0 < b1; i0 += 8 * kSelThreads) {
        uint32_t kk[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {   // eight keys per thread and step: the loads (L2 or HBM) are in flight together
          const int i = i0 + u * kSelThreads;
          kk[u] = key(min(i, b1 - 1));   // unconditional: the loads of the step are issued together
          kk[u] = i < b1 ? kk[u] : 0u;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (kk[u] != 0u && (kk[u] & mask) == prefix) atomicAdd(&sc.hist[warp][(kk[u] >> shift) & 255u], 1u);
      }
      __syncthreads();
      {   // bin tid of this block, over its warps, into the cluster's histogram
        uint32_t v = 0;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) {
          v += sc.hist[w][tid];
          sc.hist[w][tid] = 0;
        }
        if (v != 0u) cs::add_remote(total0 + static_cast<uint32_t>(tid) * 4u, v);
      }
      cs::sync();
      if (me == 0) {
        // thread t takes bin 255 - t; the block scans the counts from the top bin down and the thread whose bin holds
        // the k-th key publishes the new prefix
        const int bin = 255 - tid;
        const uint32_t cnt = sc.total[bin];
        sc.total[bin] = 0;
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += v;
        }
        if (lane == 31) sc.warp_gt[warp] = incl;
        __syncthreads();
        uint32_t before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) {
          const uint32_t v = sc.warp_gt[w];
          before += w < warp ? v : 0u;
          total += v;
        }
        incl += before;
        const uint32_t excl = incl - cnt;
        const uint32_t remaining = shift == 24 ? static_cast<uint32_t>(k > 0 ? k : 0) : sc.remaining;
        if (shift == 24 && tid == 0) {
          sc.n_valid = total;
          sc.take_all = (static_cast<int>(total) <= k || k <= 0) ? 1u : 0u;
        }
        __syncthreads();   // (remaining was read before anybody overwrites it)
        if (excl < remaining && remaining <= incl) {   // exactly one thread, unless everything is taken anyway
          sc.prefix = prefix | (static_cast<uint32_t>(bin) << shift);
          sc.remaining = remaining - excl;
        }
      }
      cs::sync();
      prefix = cs::load_remote(pub0);
      if (shift == 24) {
        n_valid = static_cast<int>(cs::load_remote(pub0 + 8));
        take_all = cs::load_remote(pub0 + 12) != 0u;
      }
      if (take_all) break;   // uniform over the cluster
      mask |= 255u << shift;
      if (shift == 0) {
        T = prefix;
        need_eq = static_cast<int>(cs::load_remote(pub0 + 4));
      }
    }
  }
  if (k <= 0 || n_valid == 0) {
    if (me == 0)
      for (int i = tid; i < k; i += kSelThreads) out[i] = -1;
    cs::sync();   // nobody leaves while its shared memory may still be addressed
    return 0;
  }

  // ---- ordered compaction: warp w of this block owns [begin, end) of the block's piece
  const int per = (((b1 - b0) + kSelWarps - 1) / kSelWarps + 31) & ~31;
  const int begin = min(b1, b0 + warp * per), end = min(b1, begin + per);
  uint32_t gt = 0, eq = 0;
  for (int i0 = begin + lane; i0 < end; i0 += 8 * 32) {
    uint32_t kk[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + 32 * u;
      kk[u] = key(min(i, end - 1));
      kk[u] = i < end ? kk[u] : 0u;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
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
  __syncthreads();
  int gt_before = 0, eq_before = 0, gt_block = 0, eq_block = 0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) {
    const int g = static_cast<int>(sc.warp_gt[w]), e = static_cast<int>(sc.warp_eq[w]);
    gt_before += w < warp ? g : 0;
    eq_before += w < warp ? e : 0;
    gt_block += g;
    eq_block += e;
  }
  const uint32_t cnt0 = cs::at_rank0(sc.cnt);
  if (tid == 0) {
    cs::store_remote(cnt0 + me * 8u, static_cast<uint32_t>(gt_block));
    cs::store_remote(cnt0 + me * 8u + 4u, static_cast<uint32_t>(eq_block));
  }
  cs::sync();
  for (uint32_t r = 0; r < me; ++r) {   // the blocks before this one
    gt_before += static_cast<int>(cs::load_remote(cnt0 + r * 8u));
    eq_before += static_cast<int>(cs::load_remote(cnt0 + r * 8u + 4u));
  }
  int out_run = gt_before + min(eq_before, need_eq);
  int eq_run = eq_before;
  const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll 1
  for (int base = begin; base < end; base += 8 * 32) {
    uint32_t kk[8], eq_mask[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + 32 * u + lane;
      kk[u] = key(min(i, end - 1));
      kk[u] = i < end ? kk[u] : 0u;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) eq_mask[u] = __ballot_sync(0xffffffffu, (kk[u] == T) && (kk[u] != 0u));
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const bool is_eq = (kk[u] == T) && (kk[u] != 0u);
      const bool sel = kk[u] > T || (is_eq && eq_run + __popc(eq_mask[u] & lt_mask) < need_eq);
      const uint32_t sel_mask = __ballot_sync(0xffffffffu, sel);
      if (sel) out[out_run + __popc(sel_mask & lt_mask)] = id(base + 32 * u + lane);
      out_run += __popc(sel_mask);
      eq_run += __popc(eq_mask[u]);
    }
  }
  const int written = min(k, n_valid);
  if (me == 0)
    for (int i = written + tid; i < k; i += kSelThreads) out[i] = -1;
  cs::sync();   // nobody leaves while its shared memory may still be addressed
  return written;
}

}  // namespace lsa
