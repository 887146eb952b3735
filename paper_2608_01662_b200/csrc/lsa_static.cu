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

// Status word of this entry point (what the workspace's first word is for the other calls): a kernel whose bounded
// wait ran out leaves LSA_ERR_TIMEOUT here.  Shared by all calls on a device, like the scratch array.
static __device__ __align__(256) int g_static_status[64];

std::mutex g_setup_mutex;
float* g_scratch_ptr[kMaxDevices];  // device address of g_static_scratch on each device, once looked up
int* g_status_ptr[kMaxDevices];     // device address of g_static_status

// Device addresses of the two arrays on `device` (which must be current).  Looked up once per device; the status
// word is cleared on that occasion.
cudaError_t symbols_for_device(int device, cudaStream_t st, float** scratch, int** status) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[device] == nullptr || g_status_ptr[device] == nullptr) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    void* q = nullptr;
    e = cudaGetSymbolAddress(&q, g_static_status);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(q, 0, sizeof(int), st);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[device] = static_cast<float*>(p);
    g_status_ptr[device] = static_cast<int*>(q);
  }
  *scratch = g_scratch_ptr[device];
  *status = g_status_ptr[device];
  return cudaSuccess;
}

// Makes `device` current for the lifetime of the object and puts the caller's device back afterwards.
struct DeviceScope {
  int previous = -1;
  bool ok = true;
  explicit DeviceScope(int device) {
    if (cudaGetDevice(&previous) != cudaSuccess) previous = -1;
    if (previous != device) ok = cudaSetDevice(device) == cudaSuccess;
    else previous = -1;   // nothing to restore
  }
  ~DeviceScope() {
    if (previous >= 0) cudaSetDevice(previous);
  }
};

}  // namespace

extern "C" int lsa_index_static(int device, void* cuda_stream, const lsa_params* p, const void* q_idx, const float* w,
                                const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0,
                                int64_t n_query, int64_t n_key, int32_t* sparse_idx, int32_t* n_sparse) {
  if (device < 0 || device >= kMaxDevices) return LSA_ERR_ARG;
  // the checks of lsa_index (parameters, pointers, ranges, 16-byte alignment) ...
  const int r = lsa::check_index_call(p, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, nullptr, 0, nullptr, 0,
                                      sparse_idx, n_sparse);
  if (r != LSA_OK) return r;
  // ... and what this entry point leaves out
  if (p->paged) return LSA_ERR_ARG;                          // contiguous caches only
  if (p->pooling != LSA_POOL_MEAN) return LSA_ERR_SHAPE;     // mean pooling only
  if (static_cast<int64_t>(p->keep_pages) * p->page > 4096) return LSA_ERR_SHAPE;   // larger budgets need workspace pieces
  if (!p->hi_enable && n_key > 4096) return LSA_ERR_SHAPE;   // so does the flat indexer over long caches
  if (n_query == 0) return LSA_OK;
  // the whole page-score matrix of the call must fit the fixed array
  const int64_t ps_ld = ((n_key + p->page - 1) / p->page + 3) / 4 * 4;
  if (n_query * ps_ld * static_cast<int64_t>(sizeof(float)) > static_cast<int64_t>(kStaticScratchBytes)) return LSA_ERR_CAPACITY;

  DeviceScope scope(device);
  if (!scope.ok) return LSA_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* scratch = nullptr;
  int* status = nullptr;
  if (symbols_for_device(device, st, &scratch, &status) != cudaSuccess) return LSA_ERR_CUDA;

  lsa::IndexArgs a{};
  a.HI = p->n_heads_idx; a.DI = p->d_idx; a.key_e4m3 = p->key_dtype == LSA_KEY_E4M3;
  a.P = p->page; a.B = p->sub_block; a.M = p->keep_pages; a.Ksp = p->k_sparse; a.S = p->k_sink; a.W = p->k_swa;
  a.hi_enable = p->hi_enable; a.paged = 0;
  a.q_idx = q_idx; a.w = w; a.k_idx = k_idx; a.k_scale = k_scale; a.kmean = kmean;
  a.q_pos0 = q_pos0; a.n_query = static_cast<int>(n_query); a.n_key = n_key;
  a.page_scores = scratch;  // no entry needs clearing: the fine stage reads only what the coarse stage wrote
  a.ps_ld = static_cast<int>(ps_ld);
  a.sparse_idx = sparse_idx; a.n_sparse = n_sparse; a.pages_out = nullptr; a.status = status;
  a.fine_parts = 1;
  int64_t launches = 0;
  cudaError_t e = cudaSuccess;
  if (p->hi_enable) e = lsa::launch_coarse_best(a, 2, st, &launches);   // the dispatch and tile grouping of lsa_index
  if (e == cudaSuccess) e = lsa::launch_fine_select(a, st, &launches);
  return e == cudaSuccess ? LSA_OK : LSA_ERR_CUDA;
}

extern "C" int lsa_index_static_status(int device, void* cuda_stream, int* device_status) {
  if (device < 0 || device >= kMaxDevices || device_status == nullptr) return LSA_ERR_ARG;
  *device_status = 0;
  DeviceScope scope(device);
  if (!scope.ok) return LSA_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* scratch = nullptr;
  int* status = nullptr;
  if (symbols_for_device(device, st, &scratch, &status) != cudaSuccess) return LSA_ERR_CUDA;
  cudaError_t e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(device_status, status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? LSA_OK : LSA_ERR_CUDA;
}
