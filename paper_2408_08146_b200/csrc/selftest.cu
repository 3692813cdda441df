// Self-test of the error path of the bounded device-side waits.
//
// The tensor-core kernels wait on shared-memory barriers with a cycle limit; when a wait runs out
// they record a timeout in the context's device status word and return.  In normal operation that
// never happens, so this kernel makes it happen in the smallest possible setting: one thread, one
// barrier that nothing arrives at, no copies or matrix multiplies in flight.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace koala {
namespace {

constexpr int E_TIMEOUT = 6;

__global__ void selftest_timeout_kernel(int *status, long long limit_cycles) {
  __shared__ uint64_t bar;
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(&bar, 0, limit_cycles);      // nobody arrives: runs out
    if (!ok && status) atomicMax(status, E_TIMEOUT);
  }
}

}  // namespace

cudaError_t selftest_timeout(Launch L, int *status, long long limit_cycles) {
  return launch_k(selftest_timeout_kernel, dim3(1), dim3(32), 0, L.st, L.pdl, status, limit_cycles);
}

}  // namespace koala
