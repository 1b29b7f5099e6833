// Cluster instantiations of the softmax kind at 2560, 3072 and 3584 columns (clusters of 10, 12 and 14 CTAs), in a translation unit of their
// own.  Behind a contraction longer than 256 such rows would otherwise take the row kernel, which computes the scores twice:
// measured (8192 rows) 8192 x 1536, K = 4096: 433 us there against 99 us on chip; 2560, K = 2048: 321 against 95.
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_softmax_more_rows_b(int form, const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock) \
  case n:                                      \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, b0, b1, cn, nst, lock, 2>(maps, p, st);
  switch (form) {  // the instantiation's row length: p.N, or the next wider one
    COMFUSE_CASE(2560, 256, 256, 5, 3, 1)
    COMFUSE_CASE(3072, 256, 256, 6, 3, 1)
    COMFUSE_CASE(3584, 256, 256, 7, 3, 1)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
