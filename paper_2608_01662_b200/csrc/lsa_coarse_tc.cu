// a1 on the 5th-generation tensor cores: coarse page scores (Eq. 9) for contiguous (prefill) caches.
//
//   I_page[t,p] = sum_j w[t,j] * sum_{n in page p} ReLU(q_I[t,j] . km[n])
//
// is a dense causal contraction km[n_sub, d_I] x q_I[(t,j), d_I]^T followed by a ReLU / head-weight /
// head-sum / sub-block-sum epilogue.  One thread block owns NG groups of 4 consecutive queries (N = 256
// = 4 queries x 64 heads per group, resident in shared memory) and streams tiles of 128 mean keys (M = 128)
// over the causal range of its last query:
//
//   warp 0      TMA producer: mean-key tiles (and the query groups once) -> 128B-swizzled shared tiles
//   warp 1      issues tcgen05.mma (M128 N256 K16, bf16 -> fp32) into one of two 256-column TMEM accumulators
//   warps 2-17  epilogue: tcgen05.ld of the finished accumulator, ReLU * w, sum over heads in-thread (one
//               thread = one mean key), sum over the sub-blocks of a page by warp shuffles, store
//
// so the epilogue of unit u overlaps the MMAs of unit u+1.  Heavy (late) query blocks are launched first.
#include "lsa_internal.h"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

constexpr int kHI = 64, kDI = 128;
constexpr int kTileM = 128;                 // mean keys per tile
constexpr int kGroupQ = 4;                  // queries per MMA group: N = kGroupQ * kHI = 256
constexpr int kAtomBytesA = kTileM * 128;   // one 64-dim column block of an A tile
constexpr int kAtomBytesB = kGroupQ * kHI * 128;
constexpr int kTileBytesA = 2 * kAtomBytesA;  // d_I = 128 = two 64-dim column blocks
constexpr int kGroupBytesB = 2 * kAtomBytesB;
constexpr int kEpiWarps = 16;               // 4 per TMEM lane quarter: one per query of the group
constexpr int kThreadsTc = 32 * (2 + kEpiWarps);
constexpr uint32_t kTmemCols = 512;

template <int NG>
struct CoarseTcSmem {
  static constexpr int kStages = NG == 1 ? 4 : 2;
  alignas(1024) uint8_t a[kStages][kTileBytesA];
  alignas(1024) uint8_t b[NG][kGroupBytesB];
  float w[NG * kGroupQ][kHI];
  alignas(8) uint64_t full[kStages], empty[kStages], q_full, acc_full[2], acc_empty[2];
  uint32_t tmem_slot;
};

template <int NG>
__global__ void __launch_bounds__(kThreadsTc, 1)
coarse_score_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_km, IndexArgs p) {
  using Smem = CoarseTcSmem<NG>;
  constexpr int NS = Smem::kStages;
  constexpr int QB = NG * kGroupQ;  // queries per block
  extern __shared__ uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // heavy blocks first: block 0 takes the last queries
  const int qb = gridDim.x - 1 - blockIdx.x;
  const int q0 = qb * QB;
  const int nq = min(QB, p.n_query - q0);
  const int64_t t_max = p.q_pos0 + q0 + nq - 1;
  const int64_t t_need = (static_cast<int64_t>(p.M) + p.S / p.P) * p.P + p.W;  // first query with more than M eligible pages
  if (t_max < t_need) return;
  if (tc::status_raised(p.status)) return;   // an earlier block of this launch gave up on a wait
  const int64_t hi_max = t_max - p.W;
  const int spp = p.P / p.B;
  const int spp_shift = 31 - __clz(spp);
  const int n_tiles = static_cast<int>(hi_max / (static_cast<int64_t>(kTileM) * p.B)) + 1;
  const int n_units = n_tiles * NG;

  // ---- set-up
  for (int i = tid; i < QB * kHI; i += kThreadsTc) {
    const int q = i / kHI;
    (&sm.w[0][0])[i] = q < nq ? p.w[static_cast<int64_t>(q0 + q) * kHI + (i % kHI)] : 0.f;
  }
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      tc::mbar_init(smem_u32(&sm.full[s]), 1);
      tc::mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    tc::mbar_init(smem_u32(&sm.q_full), 1);
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.acc_full[b]), 1);
      tc::mbar_init(smem_u32(&sm.acc_empty[b]), kEpiWarps / 2);
    }
    tc::fence_mbar_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemCols);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;

  if (warp == 0) {
    // ================= producer =================
    if (lane == 0) {
      tc::mbar_expect_tx(smem_u32(&sm.q_full), NG * kGroupBytesB);
      for (int g = 0; g < NG; ++g)
        for (int a = 0; a < 2; ++a)
          tc::tma_load_2d(smem_u32(sm.b[g]) + a * kAtomBytesB, &map_q, a * 64, (q0 + g * kGroupQ) * kHI, smem_u32(&sm.q_full));
      for (int k = 0; k < n_tiles; ++k) {
        const int s = k % NS;
        if (!tc::mbar_wait(smem_u32(&sm.empty[s]), ((k / NS) & 1) ^ 1, p.status)) break;
        tc::mbar_expect_tx(smem_u32(&sm.full[s]), kTileBytesA);
        for (int a = 0; a < 2; ++a)
          tc::tma_load_2d(smem_u32(sm.a[s]) + a * kAtomBytesA, &map_km, a * 64, k * kTileM, smem_u32(&sm.full[s]));
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16(kTileM, kGroupQ * kHI, 0, 0);
      bool ok = tc::mbar_wait(smem_u32(&sm.q_full), 0, p.status);
      for (int k = 0; k < n_tiles && ok; ++k) {
        const int s = k % NS;
        ok = tc::mbar_wait(smem_u32(&sm.full[s]), (k / NS) & 1, p.status);
        for (int g = 0; g < NG && ok; ++g) {
          const int u = k * NG + g, buf = u & 1;
          ok = tc::mbar_wait(smem_u32(&sm.acc_empty[buf]), ((u >> 1) & 1) ^ 1, p.status);
          if (!ok) break;
          tc::fence_after_sync();
          const uint32_t d = tmem_base + buf * 256;
#pragma unroll
          for (int a = 0; a < 2; ++a) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t da = tc::smem_desc_sw128(smem_u32(sm.a[s]) + a * kAtomBytesA + kk * 32, 16, 1024);
              const uint64_t db = tc::smem_desc_sw128(smem_u32(sm.b[g]) + a * kAtomBytesB + kk * 32, 16, 1024);
              tc::umma_ss(d, da, db, idesc, (a | kk) != 0);
            }
          }
          if (g == NG - 1) tc::umma_commit(smem_u32(&sm.empty[s]));  // the stage is free once these MMAs are done
          tc::umma_commit(smem_u32(&sm.acc_full[buf]));
        }
      }
    }
  } else {
    // ================= epilogue =================
    // Two sets of 8 warps: set 0 drains accumulator 0 (even units), set 1 accumulator 1 (odd units), so a warp
    // has two unit periods for its load -> math -> reduce -> store chain.  Within a set, warp (quarter, half)
    // owns TMEM lanes 32*quarter.. and the head columns of queries 2*half, 2*half+1 of the group.
    const int ew = warp - 2;
    const int set = ew >> 3;
    const int quarter = warp & 3;
    const int half = (ew >> 2) & 1;
    const int row = 32 * quarter + lane;    // mean key within the tile
    bool ok = true;
    for (int u = set; u < n_units && ok; u += 2) {
      const int k = u / NG, g = u % NG;
      ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.acc_full[set]), (u >> 1) & 1, p.status));
      if (!ok) break;
      tc::fence_after_sync();
      const int64_t page = (static_cast<int64_t>(k) * kTileM + row) >> spp_shift;   // spp is a power of two
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + set * 256 + half * 2 * kHI;
      const int ql0 = g * kGroupQ + half * 2;
      float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
      {
        uint32_t v[64];
        tc::tmem_ld64(taddr, v);
        tc::tmem_ld_wait();
        const float4* w4 = reinterpret_cast<const float4*>(&sm.w[ql0][0]);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float4 ww = w4[j];
          a0 = fmaf(ww.x, fmaxf(__uint_as_float(v[4 * j + 0]), 0.f), a0);
          a1 = fmaf(ww.y, fmaxf(__uint_as_float(v[4 * j + 1]), 0.f), a1);
          a0 = fmaf(ww.z, fmaxf(__uint_as_float(v[4 * j + 2]), 0.f), a0);
          a1 = fmaf(ww.w, fmaxf(__uint_as_float(v[4 * j + 3]), 0.f), a1);
        }
      }
      {
        uint32_t v[64];
        tc::tmem_ld64(taddr + kHI, v);
        tc::tmem_ld_wait();
        // the rest of the accumulator is in registers: hand the TMEM buffer back before the arithmetic
        tc::fence_before_sync();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(smem_u32(&sm.acc_empty[set]));
        const float4* w4 = reinterpret_cast<const float4*>(&sm.w[ql0 + 1][0]);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float4 ww = w4[j];
          b0 = fmaf(ww.x, fmaxf(__uint_as_float(v[4 * j + 0]), 0.f), b0);
          b1 = fmaf(ww.y, fmaxf(__uint_as_float(v[4 * j + 1]), 0.f), b1);
          b0 = fmaf(ww.z, fmaxf(__uint_as_float(v[4 * j + 2]), 0.f), b0);
          b1 = fmaf(ww.w, fmaxf(__uint_as_float(v[4 * j + 3]), 0.f), b1);
        }
      }
      float acc0 = a0 + a1, acc1 = b0 + b1;
      // sum over the sub-blocks of a page: spp (8, 16 or 32) adjacent lanes
      for (int off = spp >> 1; off > 0; off >>= 1) {
        acc0 += __shfl_xor_sync(0xffffffffu, acc0, off);
        acc1 += __shfl_xor_sync(0xffffffffu, acc1, off);
      }
      if ((lane & (spp - 1)) == 0) {
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          const int ql = ql0 + qq;
          const int64_t t = p.q_pos0 + q0 + ql;
          if (ql < nq && page * p.P <= t - p.W)
            p.page_scores[static_cast<int64_t>(q0 + ql) * p.ps_ld + page] = qq ? acc1 : acc0;
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

// ---- host side: tensor maps -----------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

bool tma_available() { return encode_tiled_fn() != nullptr; }

// bf16 matrix [rows, 128] row-major, box = 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
bool make_map_bf16_128(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {128, rows};
  const cuuint64_t strides[1] = {256};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map_u8_128(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {128, rows};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {128, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 matrix [rows, cols] row-major (cols a multiple of 64), box = 64 columns x box_rows rows, 128-byte swizzle.
bool make_map_bf16_rows(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            box_rows == 1 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

template <int NG>
cudaError_t launch_tc(const IndexArgs& a, cudaStream_t st, int64_t* n_launch) {
  CUtensorMap map_q, map_km;
  const uint64_t n_sub = static_cast<uint64_t>((a.n_key + a.B - 1) / a.B);
  if (!make_map_bf16_128(&map_q, a.q_idx, static_cast<uint64_t>(a.n_query) * kHI, kGroupQ * kHI) ||
      !make_map_bf16_128(&map_km, a.kmean, n_sub, kTileM))
    return cudaErrorInvalidValue;
  const size_t smem = sizeof(CoarseTcSmem<NG>) + 1024;
  auto kernel = coarse_score_tc_kernel<NG>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int QB = NG * kGroupQ;
  const int blocks = (a.n_query + QB - 1) / QB;
  kernel<<<blocks, kThreadsTc, smem, st>>>(map_q, map_km, a);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace

bool coarse_tc_supported(const IndexArgs& a) {
  return a.HI == kHI && a.DI == kDI && !a.paged && (reinterpret_cast<uintptr_t>(a.q_idx) & 15u) == 0 &&
         (reinterpret_cast<uintptr_t>(a.kmean) & 15u) == 0 && tma_available();
}

cudaError_t launch_coarse_tc(const IndexArgs& a, int groups, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  return groups == 2 ? launch_tc<2>(a, st, n_launch) : launch_tc<1>(a, st, n_launch);
}

}  // namespace lsa
