// Diagnostics entry points that are not part of the method.
#include "sm100.cuh"

namespace vmoba {

// One CTA waits, with the library's bounded wait, on an mbarrier that nothing ever arrives at: the wait gives up
// after `polls` polls, records VMOBA_ERR_TIMEOUT, and every later wait of the CTA gives up after a few polls, so
// the kernel ends by itself.  out[0] counts the waits that gave up, out[1] is set when the kernel's last
// instruction is reached.
__global__ void __launch_bounds__(64) wait_timeout_kernel(int32_t* status, uint32_t polls, int32_t* out) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  __shared__ int gave_up;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    sm100::fence_barrier_init();
    abort_flag = 0;
    gave_up = 0;
  }
  __syncthreads();
  volatile int* af = &abort_flag;
  // first wait: phase 0 never completes
  if (!sm100::mbar_wait_polls(&bar, 0, af, status, polls)) atomicAdd(&gave_up, 1);
  __syncthreads();
  // a later wait of the same CTA: drains after a few polls because the abort flag is set
  if (!sm100::mbar_wait_polls(&bar, 0, af, status, polls)) atomicAdd(&gave_up, 1);
  __syncthreads();
  if (threadIdx.x == 0 && out) { out[0] = gave_up; out[1] = 1; }
}

}  // namespace vmoba

extern "C" int vmoba_debug_wait_timeout(int32_t* dev_status, uint32_t polls, int32_t* out2_or_null, void* stream) {
  if (!dev_status || polls == 0 || polls > (1u << 16)) return VMOBA_ERR_ARG;
  vmoba::wait_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(dev_status, polls, out2_or_null);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}
