// Instantiations of the fused kernel for  P = softmax(alpha*A.B + mask)  over the last dimension
// (ReduceMode softmax of Sec. 5; the attention-score pattern of Sec. 6.1).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_softmax(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
  // Short K: recomputing a score chunk is cheaper than keeping the row block on-chip across a cluster.
  // COMFUSE_SOFTMAX_CLUSTER=1 forces the cluster kernel where it has an instantiation (for comparisons).
  static const bool force_cluster = std::getenv("COMFUSE_SOFTMAX_CLUSTER") != nullptr;
  if (softmax_rows_supported(p) && !force_cluster) return supported_only ? cudaSuccess : launch_softmax_rows(maps, p, st);
#define COMFUSE_CASE(n, b0, b1, cn, nst, epw) \
  case n:                                     \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, b0, b1, cn, nst, 0, epw>(maps, p, st);
  // The softmax passes are latency-bound on few warps and need few registers: four epilogue warps per lane quarter.
  switch (p.N) {
    COMFUSE_CASE(256, 256, 0, 1, 3, 4)
    COMFUSE_CASE(512, 256, 256, 1, 2, 4)
    COMFUSE_CASE(1024, 256, 256, 2, 2, 4)
    COMFUSE_CASE(2048, 256, 256, 4, 2, 4)
    COMFUSE_CASE(4096, 256, 256, 8, 2, 4)
    default:
      // Long K and a row length without a cluster instantiation -- above all rows wider than the largest cluster holds
      // (N > 4096): the row kernel's statistics pass followed by a second MainLoop pass takes any N.  It pays the
      // GEMM twice, which is still less than writing and re-reading the scores.
      if (p.N >= 64) return supported_only ? cudaSuccess : launch_softmax_rows(maps, p, st);
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
