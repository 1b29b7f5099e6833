// Parameter block and launcher of the fused back-to-back GEMM kernel (plain data).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace comfuse {

struct B2bParams {
  int M, K, N1, N2;
  int mblocks, mpairs;  // 128-row blocks and pairs of them (per batch)
  int batch;            // attention form: X, W1, W2, O are [batch, ., .]; MLP form: 1
  int mode;             // 0: F = GELU(. + b1), tail = + b2 + X, LayerNorm; 1: F = softmax(alpha * .), tail = none;
                        // 2: F = ReLU(. + b1), tail = ReLU(. + b2) (the streamed-K kernel)
  float alpha;          // attention form: scale of the scores
  int keys_row_major;   // attention form: W1 is [batch, N1, K] (K-major tensor-core operand) instead of [batch, K, N1]
  float eps;
  const uint16_t* X;  // also the residual of the tail
  const uint16_t* b1;
  const uint16_t* b2;
  const uint16_t* gamma;
  const uint16_t* beta;
  uint16_t* O;
  unsigned int* status;
  unsigned long long timeout_ns;
  unsigned long long* trace;  // phase timestamps of CTA 0 (builds with -DCOMFUSE_TRACE only), else null
  int trace_flags;            // tracing builds: experiment switches
};

bool b2b_fused_supported(int K, int N1, int N2, int mode);
// the attention form (b2b_gemm.cu)
cudaError_t launch_b2b_fused(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st);
// the MLP form (GELU, + b2 + X, LayerNorm) with the four stages on warps of their own (b2b_mlp.cu)
bool b2b_mlp_supported(int K, int N1, int N2);
cudaError_t launch_b2b_mlp(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st);
// the ReLU MLP form with K streamed through the first GEMM (b2b_stream.cu)
bool b2b_stream_supported(int K, int N1, int N2);
cudaError_t launch_b2b_stream(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st);

}  // namespace comfuse
