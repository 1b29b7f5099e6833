// Plain bf16 GEMM (fp32 accumulate, bf16 result written to global memory): the first half of the in-library
// unfused path that the fused kernels are timed against (the materialisation boundary of Sec. 1).
#include <cstdlib>

#include "fused_launch.cuh"

namespace comfuse {

cudaError_t launch_plain_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, FusedParams p, cudaStream_t st) {
  static const bool single_cta = std::getenv("COMFUSE_SINGLE_CTA_MMA") != nullptr;  // bring-up: the 1-CTA UMMA kernel
  if (single_cta) {
    constexpr int BN = 512;
    p.nblocks = (p.N + BN - 1) / BN;
    p.total_tiles = p.batch * p.mblocks * p.nblocks;
    return launch_fused_instance<EPI_NONE, 256, 2, 1, 4>(tmA, tmB, p, st);
  }
  // 256 x 256 tile per CTA pair, two accumulator buffers: the store epilogue overlaps the next tile's MainLoop
  constexpr int BN = 256;
  p.nblocks = (p.N + BN - 1) / BN;
  return launch_pair_instance<EPI_NONE, 256, 0, 1, 2, 6>(tmA, tmB, p, st);
}

}  // namespace comfuse
