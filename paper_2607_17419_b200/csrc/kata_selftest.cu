// Test-only entry point: runs the two bounded waits of the tensor-core kernels on a barrier that nobody arrives at,
// so that the time-out path (error status written, clean return, context still usable) can be checked on a GPU
// without a fault, a trap or an unbounded wait.  One CTA of one warp; no TMEM is allocated and no MMA or TMA is in
// flight, so there is nothing to drain when the waits give up.
#include <cuda_runtime.h>

#include "../../include/kata.h"
#include "kata_selftest.h"
#include "kata_umma.cuh"

namespace kata {
namespace {

// report[0] = 1 if the time-bounded wait gave up, report[1] = 1 if the poll-bounded wait gave up,
// report[2] = the abort flag as the other waiters of a kernel would see it; then the wait on a flag in global memory
// (report[7] is the flag: it must be 0 on entry): report[3] = 1 if the wait for a flag nobody sets gave up (2 ms limit),
// report[4] = 1 if the wait returned once this thread had published the flag, report[5] = 1 if the wait on the
// poisoned flag gave up, report[6] = 1 if it did so at once (well inside its 2 s limit).
__global__ void __launch_bounds__(32) selftest_wait_kernel(int* device_status, int* report, unsigned max_polls) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    umma::mbar_init(&bar, 1);
    umma::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool timed = umma::wait_or_abort(&bar, 0, &abort_flag);                      // 0.1 s limit
    const bool polled = umma::wait_or_abort_polls(&bar, 0, &abort_flag, max_polls);    // max_polls tries of <= 1 us
    if (report != nullptr) {
      report[0] = timed ? 0 : 1;
      report[1] = polled ? 0 : 1;
      report[2] = abort_flag;
      int* flag = report + 7;
      int aborted = 0;                                     // a fresh abort flag per wait: a raised one ends a wait early
      const bool nobody = umma::wait_flag(flag, umma::kFlagLocal, &aborted, 2000000u);
      umma::publish_flag(flag, umma::kFlagLocal);
      aborted = 0;
      const bool published = umma::wait_flag(flag, umma::kFlagLocal, &aborted, 2000000u);
      umma::publish_flag(flag, umma::kFlagPoison);
      aborted = 0;
      unsigned t0, t1;
      asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t0));
      const bool poisoned = umma::wait_flag(flag, umma::kFlagAnchor, &aborted);
      asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t1));
      report[3] = nobody ? 0 : 1;
      report[4] = published ? 1 : 0;
      report[5] = (!poisoned && aborted) ? 1 : 0;
      report[6] = t1 - t0 < 1000000u ? 1 : 0;
    }
    if ((!timed || !polled) && device_status != nullptr) atomicExch(device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  }
}

}  // namespace
}  // namespace kata

extern "C" int kata_selftest_wait_timeout(int* device_status, int* report, unsigned max_polls, void* stream) {
  if (max_polls == 0 || max_polls > (1u << 20)) return KATA_ERR_INVALID_ARG;
  kata::selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(device_status, report, max_polls);
  return cudaGetLastError() == cudaSuccess ? KATA_OK : KATA_ERR_CUDA;
}
