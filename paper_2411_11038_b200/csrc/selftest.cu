// Self-test of the bounded in-kernel wait.  Every device-side wait of the library goes through
// ptx::mbar_wait, which gives up after a wall-clock limit and lets the caller report
// EFQAT_DEV_WAIT_TIMEOUT instead of spinning.  This kernel makes exactly that happen in the
// most harmless setting there is: one warp, one shared-memory mbarrier that nobody ever
// arrives on, no bulk copy in flight and no tensor memory held.  The wait runs out after
// limit_ns, the status word is set and the kernel returns normally.
#include "internal.h"
#include "ptx.cuh"

namespace efqat {

__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
  }
  __syncwarp();
  if (threadIdx.x == 0 && !ptx::mbar_wait(&bar, 0, limit_ns)) record_status(status, EFQAT_DEV_WAIT_TIMEOUT);
}

void launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st) {
  count_launches(1);
  wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns);
}

}  // namespace efqat
