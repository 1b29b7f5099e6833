// Host-side helpers shared by the translation units of the library: tensor-map encoding through the
// driver entry point (no link-time dependency on libcuda), per-device facts, launch accounting.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "comfuse.h"
#include "fused_params.h"

namespace comfuse {

struct DeviceInfo {
  int device = -1;
  int cc_major = 0;
  int sm_count = 0;
  unsigned int* status_word = nullptr;  // device address of the module's status word
};

// Facts about the current device (cached per device).  Returns nullptr if a CUDA call fails.
const DeviceInfo* current_device_info();

void count_launch();
// Kernels are launched with programmatic stream serialization (their set-up overlaps the previous kernel's tail; they
// wait for that kernel before touching global memory) unless COMFUSE_PDL=0.
bool programmatic_launch_enabled();
// Cross-CTA aggregation mode of the row statistics: COMFUSE_REDUCE_MODE=leader, default all-to-all.
bool leader_reduce_enabled();

// Encode a 3-D bf16 tiled tensor map with 128-byte swizzle: dims/strides innermost first; strides in BYTES for
// dims 1 and 2; box = {64, box_rows, 1}.
bool encode_tmap_bf16_3d(CUtensorMap* out, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                         uint64_t stride2_bytes, uint32_t box_rows);

// Tensor maps of one GEMM -> subgraph call: operands A [batch, M, K] and B [batch, K, N], residual R and output Y
// [batch, M, N]; all bf16, 128-byte swizzle, boxes of 64 elements by 128 rows (A, R), 64 rows (B) or 32 rows (Y: one
// epilogue warp's box).
struct GemmMaps {
  CUtensorMap A, B, R, Y;
};

// Launchers implemented one per translation unit.  Each returns cudaSuccess or the launch error, and
// cudaErrorInvalidValue if no instantiation covers (N, kind).  `supported_only` asks whether an instantiation
// exists without launching.
cudaError_t launch_fused_layernorm(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
cudaError_t launch_fused_rmsnorm_max(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
cudaError_t launch_fused_norm_more_rows(int epi, const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
// Epilogue = the stage program in p.program, interpreted on-chip (N in {256, 512, 768, 1024, 2048, 4096}).
cudaError_t launch_fused_program(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
// The same kernel with p.program compiled in (generated at run time, cached per program structure and N).  `launch` =
// false stops after the compilation.  cudaErrorInvalidValue: no instantiation for N, or the compiler is unavailable / failed.
cudaError_t launch_compiled_program(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only, bool launch);
comfuse_status_t program_compiler_status(const char** why);
// Rows wider than the largest cluster (16 CTAs x 256 columns): LayerNorm / RMSNorm kinds run per 4096-column block and a
// second kernel merges the blocks' statistics (the wide-row fallback).  Returns the number of blocks, 0 = not a wide row.
constexpr int kWideRowBlock = 4096;
// The same two-kernel form for rows that WOULD fit a cluster (N <= 4096), cut into narrower column blocks: clusters of 16
// CTAs occupy 112 of the 148 SMs and leave tensor memory no room to overlap a tile's epilogue with the next MainLoop, so
// for long K the detour through one fp16 copy of the row can be the faster path.  `split_row_block` = the block width
// chosen for (epi, N, K), 0 = keep the row on chip.
// The on-chip form a LayerNorm / RMSNorm row of N columns runs on: N itself where it has one, else the next wider one when
// at most a quarter of it would be masked columns (the columns from N on then hold exact zeros, and the kernel takes its
// statistic over N), else 0 (two kernels).
inline int norm_on_chip_form(int N) {
  if (N == 1280 || N == 1536 || N == 1792) return 0;  // forms of their own, with rules of their own (split_row_block)
  for (int f : {256, 512, 768, 1024, 2048, 4096})
    if (N <= f) return (N == f || 4 * N > 3 * f) ? f : 0;
  return 0;
}
int split_row_block(int epi, int N, int K, long long row_pairs);  // row_pairs = batch * ceil(M / 256): how many tiles a row length gives
// column block width of the two-kernel form (0 = one kernel) and the number of blocks per row
inline int wide_row_block(int epi, int N, int K, long long row_pairs) {
  if (epi != EPI_LN && epi != EPI_RMS_MAX) return 0;
  const int narrow = N <= 16 * kWideRowBlock ? split_row_block(epi, N, K, row_pairs) : 0;
  if (N > kWideRowBlock && narrow == 0) return (N % kWideRowBlock == 0 && N <= 16 * kWideRowBlock) ? kWideRowBlock : 0;
  return narrow;
}
inline int wide_row_blocks(int epi, int N, int K, long long row_pairs) {
  const int w = wide_row_block(epi, N, K, row_pairs);
  return w ? (N + w - 1) / w : 0;
}
cudaError_t launch_fused_softmax(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
cudaError_t launch_fused_softmax_more_rows_a(int form, const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
cudaError_t launch_fused_softmax_more_rows_b(int form, const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only);
// Short-K row softmax (pairs of CTAs, score chunks computed twice instead of exchanged across a cluster).
bool softmax_rows_supported(const FusedParams& p);
cudaError_t launch_softmax_rows(const GemmMaps& maps, FusedParams p, cudaStream_t st);
// Plain GEMM, Z = bf16(A.B) through maps.Y, any N that is a multiple of 8.
cudaError_t launch_plain_gemm(const GemmMaps& maps, FusedParams p, cudaStream_t st);
// Y = act(alpha * A.B + bias) with the plain GEMM's tiling; p.activation = comfuse_op_t of the unary node, 0 = none.
cudaError_t launch_gemm_elementwise(const GemmMaps& maps, FusedParams p, cudaStream_t st);

}  // namespace comfuse

#include "comfuse.h"

namespace comfuse {
// Y = stage program(A . B) with the on-chip interpreter (EPI_PROGRAM).  `vecs` = the up to three row-vector parameters
// the program's CHO_ROWVEC operands index, `residual` = its full-tensor parameter or null.  `query_only`: just say
// whether an instantiation exists for N (no device is touched).
comfuse_status_t run_fused_program(int batch, int M, int N, int K, long long lda, long long ldb, long long ldy, long long batch_stride_a,
                                   long long batch_stride_b, long long batch_stride_y, const void* A, const void* B, void* Y,
                                   const StageProgram& prog, const void* const vecs[3], const void* residual, long long ldr,
                                   cudaStream_t st, bool query_only, bool b_nk = false, bool compiled = false);
// Compiles the kernel run_fused_program(..., compiled = true) would launch for this program and N (no device needed).
comfuse_status_t prepare_compiled_program(int N, const StageProgram& prog);
// Y = act(alpha * A . B + bias) (reduction-free epilogue), any N that is a multiple of 8; bias may be null.
comfuse_status_t run_gemm_elementwise(int batch, int M, int N, int K, long long lda, long long ldb, long long ldy, long long batch_stride_a,
                                      long long batch_stride_b, long long batch_stride_y, const void* A, const void* B, void* Y,
                                      const void* bias, float alpha, int activation, cudaStream_t st, bool b_nk = false);
// Z = bf16(A . B), dense [batch, M, N] (ld = N), with the plain tensor-core GEMM kernel; arguments already validated.
comfuse_status_t gemm_to_bf16(int batch, int M, int N, int K, long long lda, long long ldb, long long batch_stride_a,
                              long long batch_stride_b, const void* A, const void* B, void* Z, cudaStream_t st, bool b_nk = false);

}  // namespace comfuse
