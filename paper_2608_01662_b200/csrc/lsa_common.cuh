// Device-side helpers shared by the liblsa kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lsa {

// ---- device status word -----------------------------------------------------------------------
// Slot 0 of the workspace: 0 = fine, otherwise the first problem a kernel recorded.
enum : int { kDevOk = 0, kDevTimeout = -5, kDevBadIndex = -7 };

__device__ __forceinline__ void report_status(int* status, int code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// A cache row number taken from a caller-given list.  Checking build (-DLSA_CHECK): a number outside [0, limit)
// other than the padding value -1 is recorded in the status word and treated as padding (the row is skipped);
// limit <= 0 = the cache's size is not known to the call (paged pools).  Normal build: the number as it is.
__device__ __forceinline__ int32_t checked_row(int32_t row, int64_t limit, int* status) {
#ifdef LSA_CHECK
  if (row < -1 || (limit > 0 && row >= limit)) {
    report_status(status, kDevBadIndex);
    return -1;
  }
#endif
  return row;
}

__host__ __device__ __forceinline__ int64_t min64(int64_t a, int64_t b) { return a < b ? a : b; }
__host__ __device__ __forceinline__ int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

// ---- small PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 zero-fills the destination.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---- shared-memory tile layout ----------------------------------------------------------------
// A tile is rows of ROW_BYTES bytes cut into 16-byte units; within each 128-byte segment the unit
// index is XORed with (row & 7), so that the 8 rows an ldmatrix touches fall into 8 different banks
// groups.  ROW_BYTES must be a multiple of 128.
template <int ROW_BYTES>
__device__ __forceinline__ uint32_t swz(int row, int unit) {
  return static_cast<uint32_t>(row * ROW_BYTES + ((unit & ~7) | ((unit ^ row) & 7)) * 16);
}

// ---- e4m3 -> bf16 (exact: an e4m3 value has 4 significant bits) ----------------------------------
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint16_t two_codes) {
  __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(two_codes), __NV_E4M3);
  float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
  return pack_bf16(f.x, f.y);
}

// 16 e4m3 codes (one uint4) -> 16 bf16 (two uint4)
__device__ __forceinline__ void e4m3x16_to_bf16(const uint4& c, uint4& lo, uint4& hi) {
  lo.x = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.x & 0xffff));
  lo.y = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.x >> 16));
  lo.z = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.y & 0xffff));
  lo.w = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.y >> 16));
  hi.x = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.z & 0xffff));
  hi.y = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.z >> 16));
  hi.z = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.w & 0xffff));
  hi.w = e4m3x2_to_bf16x2(static_cast<uint16_t>(c.w >> 16));
}

// ---- bf16 query heads as e5m2 planes (B operand of FP8 MMAs against e4m3 key codes) -------------------
// A head is scaled by 2^S so that its largest element lies in [2^14, 2^15); then x = p1 + p2 + p3 with p1 = e5m2(x),
// p2 = e5m2(x - p1), p3 = e5m2(x - p1 - p2), every difference exact: a bf16 value has 8 significant bits, a plane
// takes 3; only an element below 2^-23 of its head's largest loses bits, and what it loses is below 2^-30 of that
// largest element (less than the rounding of the fp32 accumulator).
__device__ __forceinline__ int e5m2_head_shift(float head_max_abs) {
  if (!(head_max_abs > 0.f)) return 0;
  const int e = static_cast<int>((__float_as_uint(head_max_abs) >> 23) & 0xffu) - 127;
  const int s = 14 - e;
  return s > 100 ? 100 : (s < -100 ? -100 : s);
}
// 16 consecutive elements of a query head, scaled, as three e5m2 planes (16 bytes each): x = p1 + p2 + p3.
__device__ __forceinline__ void split_e5m2x16(const float (&x)[16], uint4& p1, uint4& p2, uint4& p3) {
  uint32_t out[3][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float2 r = make_float2(x[2 * j], x[2 * j + 1]);
    uint32_t c[3];
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      const __nv_fp8x2_storage_t v = __nv_cvt_float2_to_fp8x2(r, __NV_SATFINITE, __NV_E5M2);   // .x in the low byte
      const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(v, __NV_E5M2);
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h));
      r.x -= f.x;   // exact: the rest has fewer significant bits than the value
      r.y -= f.y;
      c[pl] = v;
    }
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) {
      if ((j & 1) == 0) out[pl][j >> 1] = c[pl];
      else out[pl][j >> 1] |= c[pl] << 16;
    }
  }
  p1 = make_uint4(out[0][0], out[0][1], out[0][2], out[0][3]);
  p2 = make_uint4(out[1][0], out[1][1], out[1][2], out[1][3]);
  p3 = make_uint4(out[2][0], out[2][1], out[2][2], out[2][3]);
}

// ---- order-preserving key of an fp32 score --------------------------------------------------------
// Larger score <-> larger key; -0 is folded onto +0; key 0 is never produced by a finite score and
// marks "absent".
__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s + 0.0f);  // -0 + 0 = +0
  if (b == 0x80000000u) b = 0;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ---- programmatic dependent launch -------------------------------------------------------------------
// A kernel launched with launch_pdl may be placed on the SMs while the previous kernel of the stream is still
// draining.  pdl_wait() returns once that kernel has completed and its writes are visible (a no-op for an ordinary
// launch); nothing an earlier kernel may have written is read, and nothing it may read is written, before it.
// pdl_launch_dependents() lets the next kernel's blocks be placed from then on.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace lsa
