// Instantiations of the fused kernel for  P = softmax(alpha*A.B + mask)  over the last dimension
// (ReduceMode softmax of Sec. 5; the attention-score pattern of Sec. 6.1).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_softmax(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst) \
  case n:                                \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, b0, b1, cn, nst>(maps, p, st);
  switch (p.N) {
    COMFUSE_CASE(256, 256, 0, 1, 3)
    COMFUSE_CASE(512, 256, 256, 1, 3)
    COMFUSE_CASE(1024, 256, 256, 2, 3)
    COMFUSE_CASE(2048, 256, 256, 4, 3)
    COMFUSE_CASE(4096, 256, 256, 8, 3)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
