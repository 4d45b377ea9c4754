// Self-test of the bounded wait every kernel of the tensor path is built on: one warp waits on an mbarrier that
// nothing will ever complete, with a limit of a few hundred polls. The wait must give up, raise the CTA's abort flag
// and let the kernel report FL_ERR_TIMEOUT through the status word and return normally (no trap, nothing in flight:
// no TMA copy and no MMA is issued here, so the context stays usable).
#include <cuda_runtime.h>

#include "../tc_ptx.cuh"
#include "flashloop.h"

namespace {

__global__ void __launch_bounds__(64) timeout_selftest_kernel(int* status, int* polls_seen) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);            // one arrival expected; nobody arrives
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x < 32) {
    // the same single-thread wait the MMA issuers use, with a small limit
    if (threadIdx.x == 0) ok = tc::mbar_wait(&bar, 0, &abort_flag, 300u);
  } else {
    // a second waiter that leaves as soon as it sees the flag the first one raised
    if (threadIdx.x == 32) ok = tc::mbar_wait(&bar, 0, &abort_flag, 1u << 20);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    *polls_seen = ok ? 0 : 1;
    if (abort_flag) atomicExch(status, (int)FL_ERR_TIMEOUT);
  }
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int fl_selftest_timeout(int* status, int* gave_up, void* stream) {
  timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, gave_up);
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
