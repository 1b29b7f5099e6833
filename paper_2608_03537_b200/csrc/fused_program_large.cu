// The stage-program instantiations of the fused kernel for N = 1024, 2048, 4096 (see fused_program.cu; split so
// that the two halves compile in parallel).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_program_large(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock) \
  case n:                                      \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_PROGRAM, b0, b1, cn, nst, lock>(maps, p, st);
  switch (p.N) {
    COMFUSE_PROGRAM_INSTANCES_LARGE(COMFUSE_CASE)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
