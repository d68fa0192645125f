// Diagnostics that compute nothing of the method: a self-test of the bounded wait every
// streaming kernel uses for its TMA data, so that the "a wait that never completes ends in a
// status code, not a hang" contract can be exercised without harming the device.
#include "ngc_common.cuh"
#include "ptx.cuh"

namespace ngc {
namespace {

// One warp.  Thread 0 waits on an mbarrier that expects one arrival which never comes; the
// bounded wait gives up after limit_ns, the kernel records NGC_DEV_TIMEOUT and returns.
__global__ void bounded_wait_selftest_kernel(uint64_t limit_ns, int32_t* dev_status, uint64_t* waited_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint64_t t0 = ptx::globaltimer_ns();
    const bool done = ptx::mbar_wait_bounded(&bar, 0, limit_ns);
    if (!done) set_dev_status(dev_status, NGC_DEV_TIMEOUT);
    if (waited_ns) *waited_ns = ptx::globaltimer_ns() - t0;
  }
}

}  // namespace
}  // namespace ngc

extern "C" int ngc_selftest_bounded_wait(uint32_t limit_us, int32_t* dev_status, uint64_t* waited_ns, ngc_stream stream) {
  NGC_API_RANGE("ngc_selftest_bounded_wait");
  using namespace ngc;
  if (!dev_status || limit_us == 0 || limit_us > 100000u) return NGC_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((uint64_t)limit_us * 1000ull, dev_status, waited_ns);
  return launch_status();
}
