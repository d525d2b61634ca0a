// A unit kernel for the error path that every bounded device-side wait shares: one thread waits, with a small
// limit, on an mbarrier that nothing ever arrives on.  The wait runs out, the thread records DEV_TIMEOUT in the
// status word and the kernel returns normally -- the context stays usable.  With `ticket` it first takes one ticket on
// a projection's group counter, which is the state a streaming CTA leaves behind when it gives up between its
// tickets and its finalize.
#include "common.cuh"
#include "kernels.h"
#include "umma.cuh"

namespace dart {

__global__ void __launch_bounds__(32) bounded_wait_probe_kernel(int limit, int* status, int* ticket) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    umma::mbar_init(&bar, 1);
    abort_flag = 0;
    umma::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (ticket != nullptr) atomicAdd(ticket, 1);
    if (!umma::mbar_wait(&bar, 0, &abort_flag, limit)) atomicExch(status, DEV_TIMEOUT);
  }
}

cudaError_t launch_bounded_wait_probe(int limit, int* status, int* ticket, cudaStream_t st) {
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(limit, status, ticket);
  return cudaGetLastError();
}

}  // namespace dart
