// Plain bf16 GEMM (fp32 accumulate, bf16 result written to global memory): the first half of the in-library
// unfused path that the fused kernels are timed against (the materialisation boundary of Sec. 1).
#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_plain_gemm(const GemmMaps& maps, FusedParams p, cudaStream_t st) {
  // 256 x 256 tile per CTA pair, two accumulator slots: the store epilogue overlaps the next tile's MainLoop
  constexpr int BN = 256;
  p.nblocks = (p.N + BN - 1) / BN;
  return launch_pair_instance<EPI_NONE, 256, 0, 1, 5>(maps, p, st);
}

// Y = act(alpha * A.B + bias): the same tiling with the activation in the store epilogue (reduction-free epilogues).
cudaError_t launch_gemm_elementwise(const GemmMaps& maps, FusedParams p, cudaStream_t st) {
  constexpr int BN = 256;
  p.nblocks = (p.N + BN - 1) / BN;
  return launch_pair_instance<EPI_ELEMENTWISE, 256, 0, 1, 5>(maps, p, st);
}

}  // namespace comfuse
