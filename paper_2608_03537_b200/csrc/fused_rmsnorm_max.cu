// Instantiations of the fused kernel for  H = GELU_tanh(alpha*A.B + bias) + R,  Y = RMSNorm(H) * g,  then the chained
// row max / argmax reduction (Sec. 2.2 MatMul + RMSNorm dataflow; Sec. 3.2 multi-stage chaining).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_rmsnorm_max(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock) \
  case n:                                      \
    return supported_only   ? cudaSuccess                                                                        \
           : p.no_activation ? launch_pair_instance<EPI_RMS_MAX_LINEAR, b0, b1, cn, nst, lock>(maps, p, st)        \
                             : launch_pair_instance<EPI_RMS_MAX, b0, b1, cn, nst, lock>(maps, p, st);
  // Two sub-tiles advance in lock step (lock = 1): the A tile is fetched once per K block for both.
  // Two-kernel form (p.wide): every cluster covers one p.wide_block-column block of the row, p.nblocks blocks per row.
  const int form = norm_on_chip_form(p.N);  // a row a little shorter than an instantiation runs on it, the surplus masked
  switch (p.wide ? p.wide_block : (form ? form : p.N)) {
    COMFUSE_CASE(256, 256, 0, 1, 5, 0)
    COMFUSE_CASE(512, 256, 256, 1, 3, 1)
    COMFUSE_CASE(768, 256, 128, 2, 4, 1)
    COMFUSE_CASE(1024, 256, 256, 2, 3, 1)
    COMFUSE_CASE(2048, 256, 256, 4, 3, 1)
    COMFUSE_CASE(4096, 256, 256, 8, 3, 1)
    default:
      return launch_fused_norm_more_rows(EPI_RMS_MAX, maps, p, st, supported_only);  // 1280, 1536, 1792
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
