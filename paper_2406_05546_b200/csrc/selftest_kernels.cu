// A check of the give-up path that every tensor-core kernel shares: a bounded wait on an mbarrier runs out, the
// kernel records STATUS_WAIT_TIMEOUT in the context's status word and returns normally, and the host reads the
// word back through ps_stats().  The probe kernel touches nothing but one barrier of its own in shared memory:
// no copy is in flight, no tensor memory is held, nothing faults or hangs.
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

__global__ void __launch_bounds__(32) wait_timeout_probe(uint32_t* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);                     // one arrival expected; nobody ever arrives
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait(&bar, 0, limit_cycles)) atomicOr(status, STATUS_WAIT_TIMEOUT);
}

}  // namespace

int launch_wait_timeout_probe(uint32_t* status, long long limit_cycles, cudaStream_t st) {
  wait_timeout_probe<<<1, 32, 0, st>>>(status, limit_cycles);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace psk
