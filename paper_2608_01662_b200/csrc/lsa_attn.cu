// Sparse attention over sink U window U sparse (Eq. 3), one softmax over the whole set, for a block
// of H heads that share every K/V row (absorbed-MQA / MLA latent).
//
// One thread block handles one query (or one split of one query's rows).  Rows are streamed in tiles
// of 64 keys through a double-buffered shared tile; S = Q K^T and O += P V run on tensor cores with an
// online softmax in fp32.  With the MLA latent the value tile is the key tile (v == k), so each cache
// row is read once.
#include "lsa_internal.h"
#include "lsa_common.cuh"

namespace lsa {

namespace {

constexpr int kAttnThreads = 256;
constexpr int kKeys = 64;  // keys per tile
constexpr float kLog2e = 1.4426950408889634f;

template <int H, int DQK, int DV, bool SEP_V>
struct AttnSmem {
  alignas(128) uint8_t q[H * DQK * 2];
  alignas(128) uint8_t k[2][kKeys * DQK * 2];
  alignas(128) uint8_t v[SEP_V ? 2 : 1][SEP_V ? kKeys * DV * 2 : 128];
  alignas(128) uint8_t p[H * kKeys * 2];
  float pmax[8 / (H / 16)][H];
  float psum[8 / (H / 16)][H];
  int32_t rowid[2][kKeys];
};

template <int H, int DQK, int DV, bool SEP_V>
__global__ void __launch_bounds__(kAttnThreads, 1) sparse_attn_kernel(AttnArgs p) {
  constexpr int MT = H / 16;        // 16-row head tiles
  constexpr int NWM = 8 / MT;       // warps per head tile
  constexpr int NTQ = 8 / NWM;      // 8-key n-tiles per warp in S = Q K^T
  constexpr int NTV = DV / 8 / NWM; // 8-dim n-tiles per warp in O += P V
  constexpr int KSQ = DQK / 16;
  constexpr int QROW = DQK * 2, VROW = DV * 2;
  static_assert(NTQ >= 1 && NTV >= 2 && NTV % 2 == 0, "shape");

  extern __shared__ __align__(128) uint8_t smem_raw[];
  auto& sm = *reinterpret_cast<AttnSmem<H, DQK, DV, SEP_V>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mt = warp % MT, grp = warp / MT;
  const int g = lane >> 2, c2 = (lane & 3) * 2;
  const int qi = blockIdx.x, split = blockIdx.y;

  // ---- this query's row list
  const int64_t t = p.paged ? static_cast<int64_t>(p.ctx_len[qi]) - 1 : p.q_pos0 + qi;
  int n_sink, n_sp, n_tot;
  int64_t win0;
  const int32_t* rows = nullptr;
  if (p.rows != nullptr) {
    rows = p.rows + static_cast<int64_t>(qi) * p.rows_ld;
    n_tot = p.n_rows[qi];
    n_sink = n_sp = 0;
    win0 = 0;
  } else {
    n_sink = static_cast<int>(min64(p.S, t + 1));
    win0 = max64(p.S, t - p.W + 1);
    n_sp = p.n_sparse[qi];
    n_tot = n_sink + n_sp + static_cast<int>(max64(0, t - win0 + 1));
  }
  const int32_t* sp = p.sparse_idx ? p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp : nullptr;
  auto row_of = [&](int i) -> int32_t {
    if (i >= n_tot) return -1;
    if (rows) return checked_row(rows[i], p.n_key, p.status);
    if (i < n_sink) return i;
    if (i < n_sink + n_sp) return checked_row(sp[i - n_sink], p.n_key, p.status);
    return static_cast<int32_t>(win0 + (i - n_sink - n_sp));
  };
  // slots of this split: whole tiles
  const int tiles_all = (n_tot + kKeys - 1) / kKeys;
  const int tiles_per = (tiles_all + p.n_split - 1) / p.n_split;
  const int tile_begin = split * tiles_per, tile_end = min(tiles_all, tile_begin + tiles_per);
  const int n_tiles = max(0, tile_end - tile_begin);

  const uint8_t* kg = reinterpret_cast<const uint8_t*>(p.k);
  const uint8_t* vg = reinterpret_cast<const uint8_t*>(p.v);
  auto issue_tile = [&](int tile, int buf) {
    constexpr int UK = DQK / 8;
    for (int e = tid; e < kKeys * UK; e += kAttnThreads) {
      const int r = e / UK, u = e % UK;
      const int32_t row = sm.rowid[buf][r];
      cp_async16(smem_u32(sm.k[buf]) + swz<QROW>(r, u), kg + (row >= 0 ? row : 0) * p.ld_k * 2 + u * 16, row >= 0 ? 16 : 0);
    }
    if constexpr (SEP_V) {
      constexpr int UV = DV / 8;
      for (int e = tid; e < kKeys * UV; e += kAttnThreads) {
        const int r = e / UV, u = e % UV;
        const int32_t row = sm.rowid[buf][r];
        cp_async16(smem_u32(sm.v[buf]) + swz<VROW>(r, u), vg + (row >= 0 ? row : 0) * p.ld_v * 2 + u * 16, row >= 0 ? 16 : 0);
      }
    }
    cp_async_commit();
  };
  auto write_rowids = [&](int tile, int buf) {
    if (tid < kKeys) sm.rowid[buf][tid] = tile < tile_end ? row_of(tile * kKeys + tid) : -1;
  };

  // ---- prologue: Q -> shared, row ids of the first two tiles, first tile in flight
  {
    constexpr int UQ = DQK / 8;
    const uint8_t* qg = reinterpret_cast<const uint8_t*>(p.q) + static_cast<int64_t>(qi) * H * DQK * 2;
    for (int e = tid; e < H * UQ; e += kAttnThreads) cp_async16(smem_u32(sm.q) + swz<QROW>(e / UQ, e % UQ), qg + e * 16, 16);
    cp_async_commit();
  }
  write_rowids(tile_begin, 0);
  write_rowids(tile_begin + 1, 1);
  __syncthreads();
  if (n_tiles > 0) issue_tile(tile_begin, 0);

  float o[NTV][4];
#pragma unroll
  for (int i = 0; i < NTV; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows g and g+8 of head tile mt
  const float zs = p.sm_scale * kLog2e;

  for (int it = 0; it < n_tiles; ++it) {
    const int tile = tile_begin + it, buf = it & 1;
    cp_async_wait<0>();
    __syncthreads();  // (1) tile in shared; everyone is done with the previous tile
    if (it + 1 < n_tiles) issue_tile(tile + 1, buf ^ 1);
    write_rowids(tile + 2, buf);  // read by the issue at the top of the next iteration

    // ---- S = Q K^T for head tile mt, keys [grp*8*NTQ, +8*NTQ)
    float s[NTQ][4];
#pragma unroll
    for (int i = 0; i < NTQ; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
    const uint32_t q_s = smem_u32(sm.q), k_s = smem_u32(sm.k[buf]);
    const int a_row = 16 * mt + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll 4
    for (int ks = 0; ks < KSQ; ++ks) {
      uint32_t a[4];
      ldmatrix_x4(a, q_s + swz<QROW>(a_row, 2 * ks + (lane >> 4)));
      if constexpr (NTQ == 1) {
        uint32_t b[2];
        ldmatrix_x2(b, k_s + swz<QROW>(grp * 8 + (lane & 7), 2 * ks + ((lane >> 3) & 1)));
        mma_bf16(s[0], a, b[0], b[1]);
      } else {
#pragma unroll
        for (int nt = 0; nt < NTQ; nt += 2) {
          uint32_t b[4];
          ldmatrix_x4(b, k_s + swz<QROW>(grp * 8 * NTQ + 8 * nt + (lane & 7) + (lane >> 4) * 8, 2 * ks + ((lane >> 3) & 1)));
          mma_bf16(s[nt], a, b[0], b[1]);
          mma_bf16(s[nt + 1], a, b[2], b[3]);
        }
      }
    }
    // ---- scale, mask the ragged tail, partial row max
    const int key_base = tile * kKeys + grp * 8 * NTQ;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < NTQ; ++nt) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int key = key_base + 8 * nt + c2 + (j & 1);
        const float z = key < n_tot ? s[nt][j] * zs : -INFINITY;
        s[nt][j] = z;
        mx[j >> 1] = fmaxf(mx[j >> 1], z);
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    if ((lane & 3) == 0) {
      sm.pmax[grp][16 * mt + g] = mx[0];
      sm.pmax[grp][16 * mt + g + 8] = mx[1];
    }
    __syncthreads();  // (2)
    float m_new[2], alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      float m = m_run[r];
#pragma unroll
      for (int w = 0; w < NWM; ++w) m = fmaxf(m, sm.pmax[w][16 * mt + g + 8 * r]);
      m_new[r] = m;  // finite: every tile holds at least one real key
      alpha[r] = exp2f(m_run[r] - m);
      m_run[r] = m;
    }
    // ---- P = exp2(S - m), partial row sums, P -> shared as bf16
    float sum[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < NTQ; ++nt) {
      const float p0 = exp2f(s[nt][0] - m_new[0]), p1 = exp2f(s[nt][1] - m_new[0]);
      const float p2 = exp2f(s[nt][2] - m_new[1]), p3 = exp2f(s[nt][3] - m_new[1]);
      const uint32_t lo = pack_bf16(p0, p1), hi = pack_bf16(p2, p3);
      sum[0] += p0 + p1;  // fp32 sums of the unrounded weights: lse stays exact to fp32
      sum[1] += p2 + p3;
      const int key = grp * 8 * NTQ + 8 * nt + c2;
      *reinterpret_cast<uint32_t*>(sm.p + swz<kKeys * 2>(16 * mt + g, key >> 3) + (key & 7) * 2) = lo;
      *reinterpret_cast<uint32_t*>(sm.p + swz<kKeys * 2>(16 * mt + g + 8, key >> 3) + (key & 7) * 2) = hi;
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      sum[r] += __shfl_xor_sync(0xffffffffu, sum[r], 1);
      sum[r] += __shfl_xor_sync(0xffffffffu, sum[r], 2);
    }
    if ((lane & 3) == 0) {
      sm.psum[grp][16 * mt + g] = sum[0];
      sm.psum[grp][16 * mt + g + 8] = sum[1];
    }
    __syncthreads();  // (3) P and the partial sums are in shared
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      float ssum = 0.f;
#pragma unroll
      for (int w = 0; w < NWM; ++w) ssum += sm.psum[w][16 * mt + g + 8 * r];
      l_run[r] = l_run[r] * alpha[r] + ssum;
    }
#pragma unroll
    for (int i = 0; i < NTV; ++i) {
      o[i][0] *= alpha[0];
      o[i][1] *= alpha[0];
      o[i][2] *= alpha[1];
      o[i][3] *= alpha[1];
    }
    // ---- O += P V for head tile mt, value dims [grp*8*NTV, +8*NTV)
    const uint32_t p_s = smem_u32(sm.p);
    const uint32_t v_s = SEP_V ? smem_u32(sm.v[buf]) : k_s;
    constexpr int VR = SEP_V ? VROW : QROW;
#pragma unroll
    for (int ks = 0; ks < kKeys / 16; ++ks) {
      uint32_t a[4];
      ldmatrix_x4(a, p_s + swz<kKeys * 2>(a_row, 2 * ks + (lane >> 4)));
      const int v_row = 16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int nt = 0; nt < NTV; nt += 2) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, v_s + swz<VR>(v_row, grp * NTV + nt + (lane >> 4)));
        mma_bf16(o[nt], a, b[0], b[1]);
        mma_bf16(o[nt + 1], a, b[2], b[3]);
      }
    }
  }

  // ---- epilogue
  const int row_lo = 16 * mt + g;
  if (p.n_split == 1) {
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + static_cast<int64_t>(qi) * H * DV;
    const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f, inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
#pragma unroll
    for (int nt = 0; nt < NTV; ++nt) {
      const int d = (grp * NTV + nt) * 8 + c2;
      *reinterpret_cast<uint32_t*>(out + row_lo * DV + d) = pack_bf16(o[nt][0] * inv0, o[nt][1] * inv0);
      *reinterpret_cast<uint32_t*>(out + (row_lo + 8) * DV + d) = pack_bf16(o[nt][2] * inv1, o[nt][3] * inv1);
    }
    if (p.lse != nullptr && grp == 0 && (lane & 3) == 0) {
      p.lse[static_cast<int64_t>(qi) * H + row_lo] = (m_run[0] + log2f(l_run[0])) / kLog2e;
      p.lse[static_cast<int64_t>(qi) * H + row_lo + 8] = (m_run[1] + log2f(l_run[1])) / kLog2e;
    }
  } else {
    // partial result: normalised fp32 output and log2-domain lse (-inf for an empty split)
    float* po = p.part_out + (static_cast<int64_t>(qi) * p.n_split + split) * H * DV;
    const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f, inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
#pragma unroll
    for (int nt = 0; nt < NTV; ++nt) {
      const int d = (grp * NTV + nt) * 8 + c2;
      *reinterpret_cast<float2*>(po + row_lo * DV + d) = make_float2(o[nt][0] * inv0, o[nt][1] * inv0);
      *reinterpret_cast<float2*>(po + (row_lo + 8) * DV + d) = make_float2(o[nt][2] * inv1, o[nt][3] * inv1);
    }
    if (grp == 0 && (lane & 3) == 0) {
      float* pl = p.part_lse + (static_cast<int64_t>(qi) * p.n_split + split) * H;
      pl[row_lo] = l_run[0] > 0.f ? m_run[0] + log2f(l_run[0]) : -INFINITY;
      pl[row_lo + 8] = l_run[1] > 0.f ? m_run[1] + log2f(l_run[1]) : -INFINITY;
    }
  }
}

// Merge the per-split partial results by their log-sum-exp (Sec. 4.1.1: online-softmax rescaling).
// One block per (query, head); thread d handles value dims d, d+blockDim, ...
__global__ void merge_splits_kernel(const float* __restrict__ part_out, const float* __restrict__ part_lse,
                                    int n_split, int H, int DV, __nv_bfloat16* __restrict__ out,
                                    float* __restrict__ lse) {
  constexpr int kMaxSplit = 16;
  const int qi = blockIdx.x, h = blockIdx.y;
  const float* pl = part_lse + static_cast<int64_t>(qi) * n_split * H + h;
  float wgt[kMaxSplit];
  float m = -INFINITY;
  for (int s = 0; s < n_split; ++s) {
    wgt[s] = pl[s * H];
    m = fmaxf(m, wgt[s]);
  }
  float den = 0.f;
  for (int s = 0; s < n_split; ++s) {
    wgt[s] = exp2f(wgt[s] - m);
    den += wgt[s];
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;
  for (int d = threadIdx.x * 4; d < DV; d += blockDim.x * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < n_split; ++s) {
      const float w = wgt[s] * inv;
      if (w > 0.f) {
        const float4 v = *reinterpret_cast<const float4*>(part_out + ((static_cast<int64_t>(qi) * n_split + s) * H + h) * DV + d);
        acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
      }
    }
    uint2 o;
    o.x = pack_bf16(acc.x, acc.y);
    o.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(out + (static_cast<int64_t>(qi) * H + h) * DV + d) = o;
  }
  if (lse != nullptr && threadIdx.x == 0) lse[static_cast<int64_t>(qi) * H + h] = (m + log2f(den)) / kLog2e;
}

// lsa_merge: parts are finished results (bf16, natural-log lse) of attention over disjoint key sets.
__global__ void merge_parts_kernel(MergeArgs a) {
  const int qi = blockIdx.x, h = blockIdx.y;
  const int64_t row = static_cast<int64_t>(qi) * a.H + h;
  float wgt[8];
  float m = -INFINITY;
  for (int s = 0; s < a.n_parts; ++s) {
    wgt[s] = a.lses[s][row];
    m = fmaxf(m, wgt[s]);
  }
  float den = 0.f;
  for (int s = 0; s < a.n_parts; ++s) {
    wgt[s] = m > -INFINITY ? __expf(wgt[s] - m) : 0.f;
    den += wgt[s];
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;
  for (int d = threadIdx.x * 2; d < a.DV; d += blockDim.x * 2) {
    float2 acc = make_float2(0.f, 0.f);
    for (int s = 0; s < a.n_parts; ++s) {
      const float w = wgt[s] * inv;
      if (w > 0.f) {
        const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(
            reinterpret_cast<const __nv_bfloat16*>(a.outs[s]) + row * a.DV + d));
        acc.x += w * v.x;
        acc.y += w * v.y;
      }
    }
    *reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(a.out) + row * a.DV + d) = pack_bf16(acc.x, acc.y);
  }
  if (a.lse != nullptr && threadIdx.x == 0) a.lse[row] = den > 0.f ? m + logf(den) : -INFINITY;
}

template <int H, int DQK, int DV, bool SEP_V>
cudaError_t launch_attn_t(const AttnArgs& a, cudaStream_t st, int64_t* n_launch) {
  const size_t smem = sizeof(AttnSmem<H, DQK, DV, SEP_V>);
  auto kernel = sparse_attn_kernel<H, DQK, DV, SEP_V>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  dim3 grid(a.n_query, a.n_split);
  kernel<<<grid, kAttnThreads, smem, st>>>(a);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace

bool attn_shape_supported(int H, int DQK, int DV) {
  return (H == 16 && DQK == 128 && DV == 128) || (H == 64 && DQK == 576 && DV == 512);
}

cudaError_t launch_merge_parts(const MergeArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  merge_parts_kernel<<<dim3(a.n_query, a.H), 128, 0, st>>>(a);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_merge(const AttnArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0 || a.n_split == 1) return cudaSuccess;
  merge_splits_kernel<<<dim3(a.n_query, a.H), 128, 0, st>>>(a.part_out, a.part_lse, a.n_split, a.H, a.DV,
                                                            reinterpret_cast<__nv_bfloat16*>(a.out), a.lse);
  ++*n_launch;
  return cudaGetLastError();
}

cudaError_t launch_attn(const AttnArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  const bool sep_v = !(a.v == a.k && a.ld_v == a.ld_k);
  if (a.H == 16) {
    return sep_v ? launch_attn_t<16, 128, 128, true>(a, st, n_launch) : launch_attn_t<16, 128, 128, false>(a, st, n_launch);
  }
  // the 64-head latent shape has no room for a separate value tile: MLA layout only
  if (sep_v) return cudaErrorInvalidValue;
  return launch_attn_t<64, 576, 512, false>(a, st, n_launch);
}

}  // namespace lsa
