// Kernel parameter block of the GEMM -> subgraph kernels (plain data, shared by host and device code).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace comfuse {

// EPI_RMS_MAX_LINEAR: the RMSNorm op list without its GELU (a kernel instantiation of its own, chosen by FusedParams::no_activation)
enum : int { EPI_NONE = 0, EPI_LN = 1, EPI_RMS_MAX = 2, EPI_SOFTMAX = 3, EPI_RMS_MAX_LINEAR = 4 };

struct FusedParams {
  int M, N, K, batch;
  int mblocks;      // ceil(M / 128)
  int mpairs;       // ceil(mblocks / 2): pairs of row blocks (CTA-pair kernels)
  int nblocks;      // column blocks of BN per row block (1 unless the epilogue is EPI_NONE)
  int total_tiles;  // batch * mblocks * nblocks
  float alpha, eps;
  int causal;
  int post_relu;      // LayerNorm kind: Y = max(Y, 0) after the affine step
  int no_activation;  // RMSNorm kind: no GELU in stage 1
  float softcap;      // softmax kind: > 0 = scaled scores pass through softcap * tanh(. / softcap)
  const uint16_t* bias;
  const uint16_t* gamma;
  const uint16_t* beta;
  const uint16_t* residual;
  long long ldr, batch_stride_r;
  uint16_t* Y;
  long long ldy, batch_stride_y;
  float* row_max;
  int* row_argmax;
  // Rows wider than one cluster (nblocks > 1 with a normalising epilogue): every cluster finishes stage 1 for its
  // column block only, stores the un-normalised values and writes the block's partial statistic of each row to
  // wide_partials[(batch * M + row) * nblocks + block]; a second kernel merges the partials and rescales in place.
  int wide;
  float2* wide_partials;
  // Cross-CTA aggregation of the row statistics (Sec. 3.1): 0 = all-to-all (every CTA sends its partial to every peer),
  // 1 = leader-follower (partials go to column range 0, which merges and sends the result back).  Same merge order,
  // hence the same bits, either way.
  int leader_reduce;
  unsigned int* status;
  unsigned long long timeout_ns;
  unsigned long long* trace;  // phase timestamps of CTA 0 (builds with -DCOMFUSE_TRACE only), else null
  int trace_flags;            // tracing builds: bit 0 = skip the output stores, bit 1 = skip the UMMAs
};

}  // namespace comfuse
