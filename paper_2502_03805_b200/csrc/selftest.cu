// Self-test of the bounded device-side wait used by the tensor-core kernels: one CTA initialises an mbarrier that
// nothing ever arrives on, waits on it with a short limit, and must come back with `false`, record CKV_ETIMEOUT in the
// status word and terminate normally (no trap, no endless spin).  The context stays usable afterwards.
#include "ckv_internal.h"
#include "sm100_ptx.cuh"

namespace ckv {
namespace {

__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns, int* observed) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ unsigned int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_addr(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = ptx::mbar_wait_bounded(ptx::smem_addr(&bar), 0, &abort_flag, limit_ns);
    *observed = ok ? 1 : 0;
    if (!ok) atomicExch(status, (int)CKV_ETIMEOUT);
  }
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(int* status_word, unsigned long long limit_ns, int* observed,
                                         cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status_word, limit_ns, observed);
  return cudaGetLastError();
}

}  // namespace ckv
