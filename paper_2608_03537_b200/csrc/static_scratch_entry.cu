// comfuse_gemm_epilogue_static_scratch: the unfused GEMM -> row-kernel path for callers that cannot hand the library
// a workspace because they cannot allocate device memory at the time of the call -- a real-time loop where cudaMalloc
// is forbidden, plug-ins that are given tensors but no allocator, or processes whose memory pool is owned by another
// component.  The intermediate bf16 GEMM result lives in a
// fixed-size array that is part of the loaded module instead.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/comfuse.h"

namespace {

// The scratch array.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[COMFUSE_STATIC_SCRATCH_BYTES];

// In host code the name `g_static_scratch` is only a handle for the runtime, not a device address; the address a
// kernel can use is looked up once per device, with that device current, and cached here.
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

comfuse_status_t scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return COMFUSE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();  // leave no sticky error behind
      return COMFUSE_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return COMFUSE_OK;
}

}  // namespace

extern "C" comfuse_status_t comfuse_gemm_epilogue_static_scratch(const comfuse_gemm_desc_t* desc, const void* A,
                                                                 const void* B, void* Y,
                                                                 const comfuse_epilogue_args_t* args, void* cuda_stream) {
  if (!desc) return COMFUSE_ERR_INVALID_ARG;
  comfuse_gemm_desc_t d = *desc;
  d.fused = 0;  // this entry point is the unfused path by definition; the fused kernels need no scratch at all
  size_t need = 0;
  comfuse_status_t s = comfuse_workspace_size(&d, &need);  // host-only validation of the description
  if (s != COMFUSE_OK) return s;
  if (need > static_cast<size_t>(COMFUSE_STATIC_SCRATCH_BYTES)) return COMFUSE_ERR_WORKSPACE;  // problem too large
  void* scratch = nullptr;
  s = scratch_for_current_device(&scratch);
  if (s != COMFUSE_OK) return s;
  // Nothing in the scratch has to start at zero: the GEMM kernel overwrites every element of the batch*M*N region
  // before the row kernel, ordered behind it on the same stream, reads it.
  return comfuse_gemm_epilogue(&d, A, B, Y, args, scratch, static_cast<size_t>(COMFUSE_STATIC_SCRATCH_BYTES), cuda_stream);
}
