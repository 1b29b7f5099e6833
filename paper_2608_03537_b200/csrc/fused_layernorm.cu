// Instantiations of the fused kernel for  Y = LayerNorm(alpha*A.B + bias + R) * gamma + beta  (Sec. 3.2, Fig. 3 case).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_layernorm(const CUtensorMap& tmA, const CUtensorMap& tmB, const FusedParams& p, cudaStream_t st,
                                   bool supported_only) {
#define COMFUSE_CASE(n, bns, nsub, cn, nst)                                                   \
  case n:                                                                                      \
    return supported_only ? cudaSuccess : launch_fused_instance<EPI_LN, bns, nsub, cn, nst>(tmA, tmB, p, st);
  switch (p.N) {
    COMFUSE_CASE(256, 128, 2, 1, 6)
    COMFUSE_CASE(512, 256, 2, 1, 4)
    COMFUSE_CASE(768, 192, 2, 2, 5)
    COMFUSE_CASE(1024, 256, 2, 2, 4)
    COMFUSE_CASE(2048, 256, 2, 4, 4)
    COMFUSE_CASE(4096, 256, 2, 8, 4)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
