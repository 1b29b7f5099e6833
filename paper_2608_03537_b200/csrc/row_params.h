// Parameter block of the unfused path's row kernels (plain data).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace comfuse {

struct RowParams {
  int batch, M, N;
  const uint16_t* Z;  // materialised GEMM result, bf16
  long long ldz, batch_stride_z;
  const uint16_t* bias;
  const uint16_t* gamma;
  const uint16_t* beta;
  const uint16_t* residual;
  long long ldr, batch_stride_r;
  const uint16_t* mask;  // additive [M, N] bf16 or nullptr
  int causal;
  float alpha, eps;
  int post_relu, no_activation;  // variants of the LayerNorm / RMSNorm op lists (see FusedParams)
  float softcap;                 // softmax: soft-cap of the scaled scores, 0 = none
  uint16_t* Y;
  long long ldy, batch_stride_y;
  float* row_max;
  int* row_argmax;
};

cudaError_t launch_row_epilogue(int kind, const RowParams& p, cudaStream_t st);
// Wide rows: merge the per-block partial statistics of each row and rescale the un-normalised row stored in p.Y in place.
// `block` = columns per block of the first kernel; the last block may be a partial one (N not a multiple of `block`)
cudaError_t launch_wide_row_finish(int kind, const RowParams& p, const float2* partials, int nblocks, int block, cudaStream_t st);
cudaError_t launch_bias_gelu(uint16_t* P, const uint16_t* bias, long long rows, int n, cudaStream_t st);

}  // namespace comfuse
