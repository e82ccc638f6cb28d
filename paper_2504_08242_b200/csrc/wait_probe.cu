// Failure-detection aid: makes a bounded device-side wait run out without harming anything.  One CTA initialises
// an mbarrier that nobody will ever arrive at and waits on it through the same bounded wait the tensor-core
// kernels use; when the limit is reached the wait gives up, the status word of the context is set and the kernel
// returns normally (no trap, no fault), exactly as a real kernel's wait would.
#include "kernels.h"
#include "tc_common.cuh"

namespace jup {

__global__ void __launch_bounds__(32) wait_probe_kernel(int* status, long long limit_cycles, int* gave_up) {
  __shared__ __align__(8) unsigned long long barrier_word;
  __shared__ int abort_flag;
  const uint32_t bar = smem_u32(&barrier_word);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool ok = mbar_wait(bar, 0, &abort_flag, status, limit_cycles);
    if (gave_up) *gave_up = ok ? 0 : 1;
  }
}

cudaError_t launch_wait_probe(int* status, long long limit_cycles, cudaStream_t st, LaunchInfo& li) {
  wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_cycles, nullptr);
  li.launches += 1;
  return cudaGetLastError();
}

}  // namespace jup
