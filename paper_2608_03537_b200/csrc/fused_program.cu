// Instantiations of the fused kernel whose epilogue is a stage program given as data (EPI_PROGRAM): the Stage-Stream
// passes over the TMEM-resident row block are interpreted from FusedParams::program (Sec. 3, Sec. 5.3).  Same tile
// shapes, cluster sizes and pipeline depths as the LayerNorm instantiations.
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_program_large(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);

cudaError_t launch_fused_program(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
  if (p.program.uses_temps) return cudaErrorInvalidValue;  // temporaries exist as registers of generated code only
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock) \
  case n:                                      \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_PROGRAM, b0, b1, cn, nst, lock>(maps, p, st);
  switch (p.N) {
    COMFUSE_PROGRAM_INSTANCES_SMALL(COMFUSE_CASE)
    default:
      return launch_fused_program_large(maps, p, st, supported_only);  // N = 1024, 2048, 4096: a translation unit of their own
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
