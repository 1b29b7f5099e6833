// comfuse_selftest_bounded_wait: exercises the bounded-wait machinery every kernel of the library relies on.  One CTA
// waits on an mbarrier that nothing will ever signal; the wait must give up after `timeout_ms`, record TIMEOUT in the
// device status word and let the kernel end normally.  Nothing faults, traps or spins forever: this is the library's
// failure-detection path run on purpose with a limit the caller chooses.
#include <cuda_runtime.h>

#include "../../include/comfuse.h"
#include "host_common.h"
#include "sm100_primitives.cuh"

namespace comfuse {
namespace {

__global__ void bounded_wait_selftest_kernel(unsigned int* status, unsigned long long timeout_ns, unsigned int* waits_done) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  const WaitCtx w{&abort_flag, status, timeout_ns};
  // the first waiter runs into the time limit; once the abort flag is set every other wait returns at once
  const bool ok0 = threadIdx.x == 0 ? mbar_wait<false>(smem_u32(&bar), 0, w) : true;
  __syncthreads();
  const bool ok1 = mbar_wait<false>(smem_u32(&bar), 0, w);
  if (!ok0 || !ok1) atomicAdd(waits_done, 1u);
}

__device__ unsigned int g_selftest_counter = 0;

// One element past the end of a 32-element array: the predicate is false, the store is skipped (checked build), or the
// predicate is compiled out and the kernel's own `false &&` keeps the store from happening (ordinary build).
__global__ void bounds_predicate_selftest_kernel(unsigned int* status, unsigned int* arr, int n) {
  const int i = n + static_cast<int>(threadIdx.x);  // always >= n
#ifdef COMFUSE_CHECKED
  if (COMFUSE_IN_BOUNDS(i < n, status)) arr[i] = 1u;
#else
  (void)status; (void)arr; (void)i;
#endif
}

}  // namespace
}  // namespace comfuse

using namespace comfuse;

extern "C" comfuse_status_t comfuse_selftest_bounded_wait(uint32_t timeout_ms, void* cuda_stream, uint32_t* expired_waits) {
  if (timeout_ms == 0 || timeout_ms > 1000) return COMFUSE_ERR_INVALID_ARG;  // keep the test short by construction
  const DeviceInfo* dev = current_device_info();
  if (!dev) return COMFUSE_ERR_CUDA;
  if (dev->cc_major != 10) return COMFUSE_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  void* counter = nullptr;
  if (cudaGetSymbolAddress(&counter, g_selftest_counter) != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (cudaMemsetAsync(counter, 0, sizeof(unsigned int), st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  count_launch();
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(dev->status_word, static_cast<unsigned long long>(timeout_ms) * 1000000ull,
                                                 static_cast<unsigned int*>(counter));
  if (cudaGetLastError() != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (expired_waits) {
    unsigned int h = 0;
    if (cudaMemcpyAsync(&h, counter, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    *expired_waits = h;
  }
  return COMFUSE_OK;
}

extern "C" comfuse_status_t comfuse_selftest_bounds_predicate(void* cuda_stream, int32_t* checked_build) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return COMFUSE_ERR_CUDA;
  if (dev->cc_major != 10) return COMFUSE_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  void* counter = nullptr;
  if (cudaGetSymbolAddress(&counter, g_selftest_counter) != cudaSuccess) return COMFUSE_ERR_CUDA;
  count_launch();
  bounds_predicate_selftest_kernel<<<1, 32, 0, st>>>(dev->status_word, static_cast<unsigned int*>(counter), 1);
  if (cudaGetLastError() != cudaSuccess) return COMFUSE_ERR_CUDA;
#ifdef COMFUSE_CHECKED
  if (checked_build) *checked_build = 1;
#else
  if (checked_build) *checked_build = 0;
#endif
  return COMFUSE_OK;
}
