// On-chip instantiations of the LayerNorm and RMSNorm kinds at three more row lengths -- 1280, 1536 and 1792 columns on
// clusters of 10, 6 and 14 CTAs -- in a translation unit of their own (compiled in parallel with the others).  Behind a
// short contraction these beat the two-kernel form, which is what such rows take otherwise (see split_row_block).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_norm_more_rows(int epi, const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock)                                                                              \
  case n:                                                                                                                   \
    if (supported_only) return cudaSuccess;                                                                                 \
    if (epi == EPI_LN) return launch_pair_instance<EPI_LN, b0, b1, cn, nst, lock>(maps, p, st);                             \
    return p.no_activation ? launch_pair_instance<EPI_RMS_MAX_LINEAR, b0, b1, cn, nst, lock>(maps, p, st)                    \
                           : launch_pair_instance<EPI_RMS_MAX, b0, b1, cn, nst, lock>(maps, p, st);
  if (p.wide || (epi != EPI_LN && epi != EPI_RMS_MAX)) return cudaErrorInvalidValue;
  switch (p.N) {
    COMFUSE_CASE(1280, 256, 0, 5, 5, 0)
    COMFUSE_CASE(1536, 256, 256, 3, 3, 1)
    COMFUSE_CASE(1792, 256, 0, 7, 5, 0)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
