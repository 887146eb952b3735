// Self-test of the bounded device-side wait: the path every tcgen05 kernel of the library takes when something it waits
// for never happens.  One block waits, with a caller-given cycle budget, on an mbarrier that nobody arrives on; the wait
// must run out, leave LSA_ERR_TIMEOUT in the status word and let the kernel end normally, so that the context stays
// usable.  No tensor memory, no MMA, no copy is involved, and nothing faults.
#include "lsa_internal.h"
#include "lsa_tc.cuh"

namespace lsa {

namespace {

__global__ void __launch_bounds__(64) selftest_wait_kernel(int* status, long long budget_cycles, int* waited_ok) {
  __shared__ alignas(8) uint64_t bar;
  if (threadIdx.x == 0) {
    tc::mbar_init(smem_u32(&bar), 1);   // one arrival expected; none will come
    tc::fence_mbar_init();
  }
  __syncthreads();
  // thread 0 serves the budget; the others poll with a long one and must be released by the raised status word
  const bool ok = tc::mbar_wait_budget(smem_u32(&bar), 0, status, threadIdx.x == 0 ? budget_cycles : tc::kWaitCycles);
  if (ok && waited_ok != nullptr) atomicAdd(waited_ok, 1);   // would mean the wait returned without an arrival
}

}  // namespace

cudaError_t launch_selftest_wait(int* status, long long budget_cycles, int* waited_ok, cudaStream_t st, int64_t* n_launch) {
  selftest_wait_kernel<<<1, 64, 0, st>>>(status, budget_cycles, waited_ok);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace lsa
