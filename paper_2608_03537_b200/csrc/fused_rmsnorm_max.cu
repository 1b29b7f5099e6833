// Instantiations of the fused kernels for  H = GELU_tanh(alpha*A.B + bias) + R,  Y = RMSNorm(H) * g,  then the chained
// row max / argmax reduction (Sec. 2.2 MatMul + RMSNorm dataflow; Sec. 3.2 multi-stage chaining).
#include <cstdlib>

#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_rmsnorm_max(const CUtensorMap& tmA, const CUtensorMap& tmB, const FusedParams& p, cudaStream_t st,
                                bool supported_only) {
  static const bool single_cta = std::getenv("COMFUSE_SINGLE_CTA_MMA") != nullptr;  // bring-up: the 1-CTA UMMA kernels
#define COMFUSE_CASE(n, b0, b1, cn, nacc, nst, sbns, snsub, scn, snst)                                   \
  case n:                                                                                                \
    if (supported_only) return cudaSuccess;                                                              \
    return single_cta ? launch_fused_instance<EPI_RMS_MAX, sbns, snsub, scn, snst>(tmA, tmB, p, st)           \
                      : launch_pair_instance<EPI_RMS_MAX, b0, b1, cn, nacc, nst>(tmA, tmB, p, st);
  switch (p.N) {
    COMFUSE_CASE(256, 256, 0, 1, 2, 6, 128, 2, 1, 6)
    COMFUSE_CASE(512, 256, 256, 1, 1, 4, 256, 2, 1, 4)
    COMFUSE_CASE(768, 256, 128, 2, 1, 5, 192, 2, 2, 5)
    COMFUSE_CASE(1024, 256, 256, 2, 1, 4, 256, 2, 2, 4)
    COMFUSE_CASE(2048, 256, 256, 4, 1, 4, 256, 2, 4, 4)
    COMFUSE_CASE(4096, 256, 256, 8, 1, 4, 256, 2, 8, 4)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
