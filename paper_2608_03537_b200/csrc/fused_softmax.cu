// Instantiations of the fused kernel for  P = softmax(alpha*A.B + mask)  over the last dimension
// (ReduceMode softmax of Sec. 5; the attention-score pattern of Sec. 6.1).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_softmax(const CUtensorMap& tmA, const CUtensorMap& tmB, const FusedParams& p, cudaStream_t st,
                                 bool supported_only) {
#define COMFUSE_CASE(n, bns, nsub, cn, nst)                                                   \
  case n:                                                                                      \
    return supported_only ? cudaSuccess : launch_fused_instance<EPI_SOFTMAX, bns, nsub, cn, nst>(tmA, tmB, p, st);
  switch (p.N) {
    COMFUSE_CASE(256, 128, 2, 1, 6)
    COMFUSE_CASE(512, 256, 2, 1, 4)
    COMFUSE_CASE(1024, 256, 2, 2, 4)
    COMFUSE_CASE(2048, 128, 2, 8, 6)
    COMFUSE_CASE(4096, 256, 2, 8, 4)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
