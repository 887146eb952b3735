// lsa_index_static: the indexer (coarse page scores, page top-M, fine scores, top-K_sparse) for callers
// that can hand over no scratch memory at all.  Its only scratch, the page-score matrix, lives in a
// fixed device array that is part of the library image.
#include "../../include/lsa.h"

#include <mutex>

#include "lsa_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = LSA_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Page scores of one call, fp32 [n_query, ceil(n_key/P) rounded up to 4].  Every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernels get the device address that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
float* g_scratch_ptr[kMaxDevices];  // device address of g_static_scratch on each device, once looked up

// Device address of the scratch array on `device` (which must be current).  Looked up once per device.
cudaError_t scratch_for_device(int device, float** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[device] == nullptr) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[device] = static_cast<float*>(p);
  }
  *out = g_scratch_ptr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" int lsa_index_static(int device, void* cuda_stream, const lsa_params* p, const void* q_idx, const float* w,
                                const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0,
                                int64_t n_query, int64_t n_key, int32_t* sparse_idx, int32_t* n_sparse) {
  if (p == nullptr || p->struct_size != sizeof(lsa_params)) return LSA_ERR_ARG;
  if (device < 0 || device >= kMaxDevices) return LSA_ERR_ARG;
  if (p->paged) return LSA_ERR_ARG;  // contiguous caches only
  if (p->pooling != LSA_POOL_MEAN) return LSA_ERR_SHAPE;  // mean pooling only
  if (p->key_dtype != LSA_KEY_BF16 && p->key_dtype != LSA_KEY_E4M3) return LSA_ERR_ARG;
  if (p->k_sink < 0 || p->k_swa < 0 || p->k_sparse < 0 || p->keep_pages <= 0 || p->sub_block <= 0) return LSA_ERR_ARG;
  if (!lsa::index_shape_supported(p->n_heads_idx, p->d_idx)) return LSA_ERR_SHAPE;
  if (p->page != 64 && p->page != 128 && p->page != 256) return LSA_ERR_SHAPE;
  if (p->page % p->sub_block != 0) return LSA_ERR_SHAPE;
  const int spp = p->page / p->sub_block;
  if (spp != 8 && spp != 16 && spp != 32) return LSA_ERR_SHAPE;
  if (static_cast<int64_t>(p->keep_pages) * p->page > 4096) return LSA_ERR_SHAPE;
  if (p->k_sparse > 4096 || p->k_sparse % 4 != 0) return LSA_ERR_SHAPE;
  if (!p->hi_enable && n_key > 4096) return LSA_ERR_SHAPE;
  if (q_idx == nullptr || w == nullptr || k_idx == nullptr || sparse_idx == nullptr || n_sparse == nullptr) return LSA_ERR_ARG;
  if (p->hi_enable && kmean == nullptr) return LSA_ERR_ARG;
  if (p->key_dtype == LSA_KEY_E4M3 && k_scale == nullptr) return LSA_ERR_ARG;
  if (n_query < 0 || n_key < 0 || q_pos0 < 0 || q_pos0 + n_query > n_key) return LSA_ERR_ARG;
  if (n_query == 0) return LSA_OK;
  // the whole page-score matrix of the call must fit the fixed array
  const int64_t ps_ld = ((n_key + p->page - 1) / p->page + 3) / 4 * 4;
  if (n_query * ps_ld * static_cast<int64_t>(sizeof(float)) > static_cast<int64_t>(kStaticScratchBytes)) return LSA_ERR_CAPACITY;

  int current = -1;
  if (cudaGetDevice(&current) != cudaSuccess || current != device) {
    if (cudaSetDevice(device) != cudaSuccess) return LSA_ERR_CUDA;
  }
  float* scratch = nullptr;
  if (scratch_for_device(device, &scratch) != cudaSuccess) return LSA_ERR_CUDA;

  lsa::IndexArgs a{};
  a.HI = p->n_heads_idx; a.DI = p->d_idx; a.key_e4m3 = p->key_dtype == LSA_KEY_E4M3;
  a.P = p->page; a.B = p->sub_block; a.M = p->keep_pages; a.Ksp = p->k_sparse; a.S = p->k_sink; a.W = p->k_swa;
  a.hi_enable = p->hi_enable; a.paged = 0;
  a.q_idx = q_idx; a.w = w; a.k_idx = k_idx; a.k_scale = k_scale; a.kmean = kmean;
  a.q_pos0 = q_pos0; a.n_query = static_cast<int>(n_query); a.n_key = n_key;
  a.page_scores = scratch;  // no entry needs clearing: the fine stage reads only what the coarse stage wrote
  a.ps_ld = static_cast<int>(ps_ld);
  a.sparse_idx = sparse_idx; a.n_sparse = n_sparse; a.pages_out = nullptr; a.status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int64_t launches = 0;
  cudaError_t e = cudaSuccess;
  if (p->hi_enable) e = lsa::launch_coarse(a, st, &launches);
  if (e == cudaSuccess) e = lsa::launch_fine_select(a, st, &launches);
  return e == cudaSuccess ? LSA_OK : LSA_ERR_CUDA;
}
