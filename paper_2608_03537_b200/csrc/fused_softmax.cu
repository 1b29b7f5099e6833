// Instantiations of the fused kernel for  P = softmax(alpha*A.B + mask)  over the last dimension
// (ReduceMode softmax of Sec. 5; the attention-score pattern of Sec. 6.1).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_softmax(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
  // Short K: recomputing a score chunk is cheaper than keeping the row block on-chip across a cluster.
  // COMFUSE_SOFTMAX_CLUSTER=1 forces the cluster kernel where it has an instantiation (for comparisons).
  static const bool force_cluster = std::getenv("COMFUSE_SOFTMAX_CLUSTER") != nullptr;
  // ... unless the problem is so small that the row kernel's CTA pairs do not fill the machine: up to 32 pairs of row blocks
  // (8192 rows) of 768 columns or more run faster on clusters, which put 4 to 16 CTAs on every pair.  Measured at 8192 rows,
  // K = 64 (row kernel / cluster kernel, us): N = 768: 22.3 / 15.2, 1024: 19.1 / 15.7, 2048 causal: 31.8 / 26.5, 4096: 59.1 / 50.7;
  // at 16384 rows the row kernel is ahead again (N = 2048 causal: 32.5 / 41.4), and far ahead once the output outgrows L2.
  // A row length between two instantiations runs on the next wider one: the columns from N on read as zeros and are
  // masked like the ones above the diagonal of a causal mask.
  static const int kForms[] = {256, 512, 768, 1024, 1280, 1536, 1792, 2048, 2560, 3072, 3584, 4096};
  int form = 0;
  for (int f : kForms)
    if (form == 0 && p.N <= f) form = f;
  const long long row_pairs = static_cast<long long>(p.batch) * ((p.M + 255) / 256);
  const bool small = row_pairs <= 32 && form >= 768 && p.N > form / 2;
  if (softmax_rows_supported(p) && !force_cluster && !small) return supported_only ? cudaSuccess : launch_softmax_rows(maps, p, st);
#define COMFUSE_CASE(n, b0, b1, cn, nst, epw) \
  case n:                                     \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, b0, b1, cn, nst, 0, epw>(maps, p, st);
  // Behind a long contraction the MainLoop is what counts: three pipeline stages with both sub-tiles in lock step (the A
  // tile fetched once per K block) and eight epilogue warps, instead of two stages and sixteen warps.  Measured: 8192 x 1024,
  // K = 1024: 24.1 us against 28.7; 8192 x 4096, K = 1024: 106.6 against 126.1; but K = 320 / 512 (causal): 39.2 / 44.9
  // against 36.4 / 43.1.  COMFUSE_SOFTMAX_STAGES=2 or 3 forces either form.
  static const char* stages_env = std::getenv("COMFUSE_SOFTMAX_STAGES");
  const bool long_k = stages_env ? stages_env[0] == '3' : p.K >= 768;
  if (long_k) {
    switch (form) {
      case 256: return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, 256, 0, 1, 5, 0, 2>(maps, p, st);
      case 512: return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, 256, 256, 1, 3, 1, 2>(maps, p, st);
      case 1024: return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, 256, 256, 2, 3, 1, 2>(maps, p, st);
      case 2048: return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, 256, 256, 4, 3, 1, 2>(maps, p, st);
      case 4096: return supported_only ? cudaSuccess : launch_pair_instance<EPI_SOFTMAX, 256, 256, 8, 3, 1, 2>(maps, p, st);
      default: break;
    }
  }
  // Else the softmax passes are latency-bound on few warps and need few registers: four epilogue warps per lane quarter.
  switch (form) {
    COMFUSE_CASE(256, 256, 0, 1, 3, 4)
    COMFUSE_CASE(512, 256, 256, 1, 2, 4)
    COMFUSE_CASE(1024, 256, 256, 2, 2, 4)
    COMFUSE_CASE(2048, 256, 256, 4, 2, 4)
    COMFUSE_CASE(4096, 256, 256, 8, 2, 4)
    case 768: case 1280: case 1536: case 1792:
      return launch_fused_softmax_more_rows_a(form, maps, p, st, supported_only);  // translation units of their own
    case 2560: case 3072: case 3584:
      return launch_fused_softmax_more_rows_b(form, maps, p, st, supported_only);
    default:
      // Long K and rows wider than the largest cluster holds (N > 4096): the row kernel's statistics pass followed by a
      // second MainLoop pass takes any N.  It pays the GEMM twice, which is still less than writing and re-reading the scores.
      if (p.N >= 64) return supported_only ? cudaSuccess : launch_softmax_rows(maps, p, st);
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
