// Self-test of the bounded waits the LM-head kernels are built on.
//
// Every mbarrier wait of k_lm_head gives up after a wall-clock limit, raises ATGRPO_ERR_TIMEOUT in
// the caller's status word and tells the rest of its CTA to leave (sm100.cuh).  In a healthy run
// no wait ever expires, so that path would stay unexercised.  This file holds one tiny kernel that
// makes it run without disturbing anything else: a single CTA with no TMA and no tensor memory
// waits on a barrier that nothing will ever arrive on, with a limit of a few milliseconds, and
// returns normally.  No trap, no fault, no unbounded loop: the context stays usable.
#include "internal.h"
#include "sm100.cuh"

namespace atgrpo {
namespace {
using namespace sm100;

// Warp 0 spins on the barrier (mbar_wait), warp 1 polls it with back-off (mbar_wait_backoff);
// whichever limit runs out first raises the status and sets the abort flag, and the other wait
// must then return false as well.  waited[0..1] = 1 for each warp whose wait returned false.
__global__ void __launch_bounds__(64) k_bounded_wait_selftest(unsigned long long limit_ns, int32_t* status,
                                                              int32_t* waited) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int s_abort;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    s_abort = 0;
    fence_mbar_init();
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;
  if (threadIdx.x == 0) {
    const bool ok = mbar_wait(b, 0, abort_flag, status, limit_ns);
    if (waited) waited[0] = ok ? 0 : 1;
  } else if (threadIdx.x == 32) {
    const bool ok = mbar_wait_backoff(b, 0, abort_flag, status, 2 * limit_ns);
    if (waited) waited[1] = ok ? 0 : 1;
  }
  __syncthreads();
}

}  // namespace
}  // namespace atgrpo

extern "C" int atgrpo_selftest_bounded_wait(int64_t limit_ns, int32_t* device_status, int32_t* waited,
                                            void* stream) {
  // the limit is kept short on purpose: the kernel holds one SM for at most twice this long
  if (limit_ns < 1000 || limit_ns > 50ll * 1000 * 1000 || device_status == nullptr)
    return ATGRPO_ERR_INVALID_ARG;
  atgrpo::k_bounded_wait_selftest<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      (unsigned long long)limit_ns, device_status, waited);
  return atgrpo::launch_ok();
}
