// Self-test of the bounded-wait mechanism every kernel of this library relies on: a wait on a
// barrier that nothing ever completes must give up after its limit, report through the status
// word and leave the context usable -- no trap, no endless spin.
#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(unsigned int* status, long long limit_cycles,
                                                                   long long* waited_cycles) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);          // one arrival expected; nobody arrives
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    ok = mbar_wait_slow(&bar, 0, &abort_flag, limit_cycles);
    if (waited_cycles) *waited_cycles = clock64() - t0;
  } else if (threadIdx.x == 32) {
    // a second role waiting on the same barrier sees the abort flag and stops as well
    ok = mbar_wait_slow(&bar, 0, &abort_flag, 1ll << 40);
  }
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag && status) atomicExch(status, STATUS_TIMEOUT_MBARRIER);
}

}  // namespace xema

extern "C" int xema_selftest_wait_timeout(void* status_dev, int64_t limit_cycles, int64_t* waited_cycles_dev,
                                          void* stream) {
  if (!status_dev || limit_cycles < 1 || limit_cycles > 4000000000ll) return XEMA_EINVAL;
  xema::wait_timeout_selftest_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      static_cast<unsigned int*>(status_dev), limit_cycles, reinterpret_cast<long long*>(waited_cycles_dev));
  return xema::check_launch();
}
