// Instantiations of the fused kernel for  Y = LayerNorm(alpha*A.B + bias + R) * gamma + beta  (Sec. 3.2, Fig. 3 case).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_fused_layernorm(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only) {
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock) \
  case n:                                      \
    return supported_only ? cudaSuccess : launch_pair_instance<EPI_LN, b0, b1, cn, nst, lock>(maps, p, st);
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
      return launch_fused_norm_more_rows(EPI_LN, maps, p, st, supported_only);  // 1280, 1536, 1792: a translation unit of their own
  }
#undef COMFUSE_CASE
}

}  // namespace comfuse
