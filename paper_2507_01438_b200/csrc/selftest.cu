// Self-test of the bounded-wait path: the kernels of this library never spin without a limit; a
// wait that runs out raises EDGELORA_STATUS_TIMEOUT in the device status word and the kernel
// returns, so that the context stays usable.  This kernel makes exactly that happen on purpose,
// harmlessly: one thread waits on a shared-memory barrier that nothing ever arrives at.
#include "internal.cuh"
#include "ptx.cuh"

namespace edgelora {

__global__ void __launch_bounds__(32) wait_selftest_kernel(uint32_t *status, long long wait_cycles) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
    if (!ptx::mbar_wait(&bar, 0, wait_cycles)) atomicOr(status, EDGELORA_STATUS_TIMEOUT);
  }
}

cudaError_t launch_wait_selftest(uint32_t *status, long long wait_cycles, cudaStream_t stream) {
  wait_selftest_kernel<<<1, 32, 0, stream>>>(status, wait_cycles);
  return cudaGetLastError();
}

}  // namespace edgelora
