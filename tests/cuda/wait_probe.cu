// Test-only kernel: shows that the library's bounded mbarrier wait gives up.
//
// Built against the product's own ptx_sm100.cuh with a small WK_WAIT_CAP, so the wait under test is the wait the
// attention kernel uses.  One thread initialises an mbarrier that expects one arrival.  With complete = 0 nobody ever
// arrives: the wait must run out of tries, return false, and the kernel records WK_DEV_TIMEOUT in the caller's status
// word and returns normally -- nothing spins forever, nothing traps, the context stays usable.  With complete = 1 the
// same thread arrives first, the wait succeeds and no bit is set.
#include "../../paper_2605_22718_b200/csrc/ptx_sm100.cuh"
#include "../../include/wk.h"

namespace {

__global__ void wait_probe_kernel(uint32_t* status, int complete, uint32_t* tries_out) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    wk::ptx::mbar_init(&bar, 1);
    wk::ptx::fence_mbar_init();
    if (complete) wk::ptx::mbar_arrive(&bar);
    const bool ok = wk::ptx::mbar_wait(&bar, 0);
    if (!ok) atomicOr(status, WK_DEV_TIMEOUT);
    *tries_out = ok ? 0u : static_cast<uint32_t>(WK_WAIT_CAP);
  }
}

}  // namespace

// status_dev, tries_out_dev: device words.  Returns the cudaError_t of the launch.
extern "C" int wk_test_wait_probe(uint32_t* status_dev, int complete, uint32_t* tries_out_dev, void* stream) {
  wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_dev, complete, tries_out_dev);
  return static_cast<int>(cudaGetLastError());
}
