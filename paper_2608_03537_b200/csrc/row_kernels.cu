// Second half of the in-library UNFUSED path: row kernels that read the materialised bf16 GEMM result back
// from global memory and run the same elementwise / reduction subgraph (the conventional execution the paper
// argues against in Sec. 1: on-chip -> off-chip -> on-chip).  One row is held in registers by a warp (N <= 1024)
// or by a 256-thread block (N <= 8192); reductions are warp shuffles plus one shared-memory step.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "host_common.h"
#include "row_params.h"

namespace comfuse {
namespace {

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  f[0] = bf_lo(u.x); f[1] = bf_hi(u.x); f[2] = bf_lo(u.y); f[3] = bf_hi(u.y);
  f[4] = bf_lo(u.z); f[5] = bf_hi(u.z); f[6] = bf_lo(u.w); f[7] = bf_hi(u.w);
}
__device__ __forceinline__ float gelu_tanh_ref(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.f + tanhf(u));
}

struct SumOp { __device__ float operator()(float a, float b) const { return a + b; } };
struct MaxOp { __device__ float operator()(float a, float b) const { return fmaxf(a, b); } };

// Reduce over the TPR threads that share a row.  TPR = 32: shuffle only.  TPR = 256: one row per block.
template <int TPR, class Op>
__device__ __forceinline__ float row_reduce(float v, Op op, float* s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = op(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  if constexpr (TPR > 32) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // previous use of s_red is over
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    v = s_red[0];
#pragma unroll
    for (int i = 1; i < TPR / 32; ++i) v = op(v, s_red[i]);
  }
  return v;
}

template <int TPR>
__device__ __forceinline__ void row_argmax_reduce(float& v, int& idx, float* s_red, int* s_idx) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, idx, o);
    if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
  }
  if constexpr (TPR > 32) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) { s_red[warp] = v; s_idx[warp] = idx; }
    __syncthreads();
    v = s_red[0]; idx = s_idx[0];
#pragma unroll
    for (int i = 1; i < TPR / 32; ++i) {
      const float ov = s_red[i];
      const int oi = s_idx[i];
      if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
    }
  }
}

template <int KIND, int TPR, int VPT>
__global__ void __launch_bounds__(256) row_epilogue_kernel(const RowParams p) {
  __shared__ float s_red[8];
  __shared__ int s_idx[8];
  constexpr int ROWS_PER_BLOCK = 256 / TPR;
  const int t = threadIdx.x % TPR;
  const long long r = static_cast<long long>(blockIdx.x) * ROWS_PER_BLOCK + threadIdx.x / TPR;  // row over batch*M
  const bool row_ok = r < static_cast<long long>(p.batch) * p.M;
  const int b = row_ok ? static_cast<int>(r / p.M) : 0;
  const int i = row_ok ? static_cast<int>(r - static_cast<long long>(b) * p.M) : 0;
  const uint16_t* z = p.Z + static_cast<long long>(b) * p.batch_stride_z + static_cast<long long>(i) * p.ldz;
  const uint16_t* res = p.residual ? p.residual + static_cast<long long>(b) * p.batch_stride_r + static_cast<long long>(i) * p.ldr : nullptr;
  uint16_t* y = p.Y + static_cast<long long>(b) * p.batch_stride_y + static_cast<long long>(i) * p.ldy;
  const int nvec = p.N >> 3;
  const float invN = 1.f / static_cast<float>(p.N);

  float x[VPT][8];
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int vi = t + v * TPR;
    const bool ok = row_ok && vi < nvec;
    float zf[8], bf[8], rf[8];
    uint4 zero = make_uint4(0, 0, 0, 0);
    unpack8(ok ? __ldg(reinterpret_cast<const uint4*>(z) + vi) : zero, zf);
    unpack8((ok && p.bias) ? __ldg(reinterpret_cast<const uint4*>(p.bias) + vi) : zero, bf);
    unpack8((ok && res) ? __ldg(reinterpret_cast<const uint4*>(res) + vi) : zero, rf);
    float mf[8];
    if constexpr (KIND == EPI_SOFTMAX) {
      unpack8((ok && p.mask) ? __ldg(reinterpret_cast<const uint4*>(p.mask + static_cast<long long>(i) * p.N) + vi) : zero, mf);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = vi * 8 + j;
      if constexpr (KIND == EPI_LN) {
        x[v][j] = ok ? fmaf(p.alpha, zf[j], bf[j]) + rf[j] : 0.f;
      } else if constexpr (KIND == EPI_RMS_MAX) {
        const float z = fmaf(p.alpha, zf[j], bf[j]);
        x[v][j] = ok ? (p.no_activation ? z : gelu_tanh_ref(z)) + rf[j] : 0.f;
      } else {
        float tv = p.alpha * zf[j];
        if (p.softcap > 0.f) tv = p.softcap * tanhf(tv / p.softcap);
        tv += mf[j];
        if (p.causal && col > i) tv = -INFINITY;
        x[v][j] = ok ? tv : -INFINITY;
      }
    }
  }

  if constexpr (KIND == EPI_LN) {
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int j = 0; j < 8; ++j) s += x[v][j];
    const float mu = row_reduce<TPR>(s, SumOp(), s_red) * invN;
    float m2 = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const bool ok = (t + v * TPR) < nvec;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float d = ok ? x[v][j] - mu : 0.f;
        m2 = fmaf(d, d, m2);
      }
    }
    const float rstd = rsqrtf(row_reduce<TPR>(m2, SumOp(), s_red) * invN + p.eps);
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const int vi = t + v * TPR;
      if (!(row_ok && vi < nvec)) continue;
      float gf[8], bf[8];
      uint4 one = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
      unpack8(p.gamma ? __ldg(reinterpret_cast<const uint4*>(p.gamma) + vi) : one, gf);
      unpack8(p.beta ? __ldg(reinterpret_cast<const uint4*>(p.beta) + vi) : make_uint4(0, 0, 0, 0), bf);
      float o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        o[j] = fmaf((x[v][j] - mu) * rstd, gf[j], bf[j]);
        if (p.post_relu) o[j] = fmaxf(o[j], 0.f);
      }
      reinterpret_cast<uint4*>(y)[vi] = make_uint4(pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
    }
  } else if constexpr (KIND == EPI_RMS_MAX) {
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int j = 0; j < 8; ++j) s = fmaf(x[v][j], x[v][j], s);
    const float rstd = rsqrtf(row_reduce<TPR>(s, SumOp(), s_red) * invN + p.eps);
    float best = -INFINITY;
    int best_col = 0x7FFFFFFF;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const int vi = t + v * TPR;
      if (!(row_ok && vi < nvec)) continue;
      float gf[8];
      uint4 one = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
      unpack8(p.gamma ? __ldg(reinterpret_cast<const uint4*>(p.gamma) + vi) : one, gf);
      float o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        o[j] = x[v][j] * rstd * gf[j];
        if (o[j] > best) { best = o[j]; best_col = vi * 8 + j; }
      }
      reinterpret_cast<uint4*>(y)[vi] = make_uint4(pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
    }
    row_argmax_reduce<TPR>(best, best_col, s_red, s_idx);
    if (row_ok && t == 0) {
      p.row_max[r] = best;
      p.row_argmax[r] = best_col;
    }
  } else {
    float m = -INFINITY;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int j = 0; j < 8; ++j) m = fmaxf(m, x[v][j]);
    m = row_reduce<TPR>(m, MaxOp(), s_red);
    const float msafe = (m == -INFINITY) ? 0.f : m;
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        x[v][j] = (x[v][j] == -INFINITY) ? 0.f : __expf(x[v][j] - msafe);
        s += x[v][j];
      }
    s = row_reduce<TPR>(s, SumOp(), s_red);
    const float inv = (s > 0.f) ? 1.f / s : 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const int vi = t + v * TPR;
      if (!(row_ok && vi < nvec)) continue;
      float o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = x[v][j] * inv;
      reinterpret_cast<uint4*>(y)[vi] = make_uint4(pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
    }
  }
}

// Second kernel of the two-kernel form: the fused kernel stored the un-normalised x (fp16, 11 significant bits) in Y and
// one partial statistic per row and column block; merge the partials in block order, rescale the row in place to bf16, and
// (RMSNorm kind) take the row maximum / lowest arg max of the normalised values.  One WARP per row: a lane keeps up to
// eight 16-byte loads in flight and the row reduce is a shuffle, so nothing waits on a block barrier.
__device__ __forceinline__ void unpack8_f16(const uint4 q4, float (&xf)[8]) {
  const uint32_t qw[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&qw[j]));
    xf[2 * j] = f.x;
    xf[2 * j + 1] = f.y;
  }
}

template <int KIND>
__global__ void __launch_bounds__(256) wide_row_finish_kernel(const RowParams p, const float2* partials, int nblocks, int block, long long rows) {
  // launched with programmatic stream serialization: everything above this line may overlap the first kernel's tail
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31;
  // rows from the last to the first: the first kernel wrote them in rising order, so the blocks that start first read what
  // is most likely still in L2
  const long long r = rows - 1 - (static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5));  // row over batch * M
  if (r < 0) return;
  const int b = static_cast<int>(r / p.M);
  const int i = static_cast<int>(r - static_cast<long long>(b) * p.M);
  uint16_t* y = p.Y + static_cast<long long>(b) * p.batch_stride_y + static_cast<long long>(i) * p.ldy;
  const float2* q = partials + r * nblocks;
  const float wb = static_cast<float>(block);                    // columns per block
  const int last = p.N - (nblocks - 1) * block;                  // valid columns of the last block (== block: none partial)
  float mu = 0.f, rstd;
  if constexpr (KIND == EPI_LN) {
    if (last == block) {
      // equal-count Chan merge: mean of the block means, M2 = sum M2_b + wb * sum (mean_b - mean)^2
      float ms = 0.f;
      for (int k = 0; k < nblocks; ++k) ms += q[k].x;
      mu = ms / static_cast<float>(nblocks);
      float m2 = 0.f;
      for (int k = 0; k < nblocks; ++k) {
        const float d = q[k].x - mu;
        m2 += q[k].y + wb * d * d;
      }
      rstd = rsqrtf(m2 / static_cast<float>(p.N) + p.eps);
    } else {
      // The last block is a partial one: the first kernel's statistic covers its `block` columns, of which block - last
      // are exact zeros (operands outside the matrix read as zero, the bias is masked).  Zeros add nothing to the sum and
      // to the sum of squares, so the statistic of the valid columns alone follows: S = wb mean', Sxx = M2' + wb mean'^2,
      // mean = S / last, M2 = Sxx - last mean^2.  Then the merge with the blocks' true counts.
      const float lf = static_cast<float>(last);
      float2 ql = q[nblocks - 1];
      const float s_last = wb * ql.x, sxx = ql.y + wb * ql.x * ql.x;
      ql.x = s_last / lf;
      ql.y = fmaxf(sxx - lf * ql.x * ql.x, 0.f);
      float ms = lf * ql.x;
      for (int k = 0; k + 1 < nblocks; ++k) ms += wb * q[k].x;
      mu = ms / static_cast<float>(p.N);
      const float dl = ql.x - mu;
      float m2 = ql.y + lf * dl * dl;
      for (int k = 0; k + 1 < nblocks; ++k) {
        const float d = q[k].x - mu;
        m2 += q[k].y + wb * d * d;
      }
      rstd = rsqrtf(m2 / static_cast<float>(p.N) + p.eps);
    }
  } else {
    float ss = 0.f;
    for (int k = 0; k < nblocks; ++k) ss += q[k].x;
    rstd = rsqrtf(ss / static_cast<float>(p.N) + p.eps);
  }
  float best = -INFINITY;
  int best_col = 0x7FFFFFFF;
  const int nvec = p.N >> 3;
  const uint4 one = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
  for (int v0 = 0; v0 < nvec; v0 += 32 * 8) {
    uint4 xq[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int vi = v0 + u * 32 + lane;
      if (vi < nvec) xq[u] = __ldcs(reinterpret_cast<const uint4*>(y) + vi);  // read once: streaming
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int vi = v0 + u * 32 + lane;
      if (vi >= nvec) continue;
      float xf[8], gf[8], bf[8], o[8];
      unpack8_f16(xq[u], xf);
      unpack8(p.gamma ? __ldg(reinterpret_cast<const uint4*>(p.gamma) + vi) : one, gf);
      unpack8((KIND == EPI_LN && p.beta) ? __ldg(reinterpret_cast<const uint4*>(p.beta) + vi) : make_uint4(0, 0, 0, 0), bf);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if constexpr (KIND == EPI_LN) {
          o[j] = fmaf((xf[j] - mu) * rstd, gf[j], bf[j]);
          if (p.post_relu) o[j] = fmaxf(o[j], 0.f);
        } else {
          o[j] = xf[j] * rstd * gf[j];
          if (o[j] > best) { best = o[j]; best_col = vi * 8 + j; }
        }
      }
      reinterpret_cast<uint4*>(y)[vi] = make_uint4(pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
    }
  }
  if constexpr (KIND == EPI_RMS_MAX) {
    row_argmax_reduce<32>(best, best_col, nullptr, nullptr);
    if (lane == 0) {
      p.row_max[r] = best;
      p.row_argmax[r] = best_col;
    }
  }
}

// S = bf16(GELU_tanh(P + b1)), in place over a dense [rows, n] bf16 matrix (unfused B2B: the intermediate epilogue).
__global__ void __launch_bounds__(256) bias_gelu_kernel(uint16_t* P, const uint16_t* bias, long long nvec_total, int nvec_row) {
  const long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (v >= nvec_total) return;
  const int vc = static_cast<int>(v % nvec_row);
  float pf[8], bf[8];
  unpack8(reinterpret_cast<const uint4*>(P)[v], pf);
  unpack8(bias ? __ldg(reinterpret_cast<const uint4*>(bias) + vc) : make_uint4(0, 0, 0, 0), bf);
  float o[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) o[j] = gelu_tanh_ref(pf[j] + bf[j]);
  reinterpret_cast<uint4*>(P)[v] = make_uint4(pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
}

template <int KIND, int TPR, int VPT>
cudaError_t launch_rows(const RowParams& p, cudaStream_t st) {
  constexpr int ROWS_PER_BLOCK = 256 / TPR;
  const long long rows = static_cast<long long>(p.batch) * p.M;
  const unsigned blocks = static_cast<unsigned>((rows + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK);
  count_launch();
  row_epilogue_kernel<KIND, TPR, VPT><<<blocks, 256, 0, st>>>(p);
  return cudaGetLastError();
}

template <int KIND>
cudaError_t dispatch_rows(const RowParams& p, cudaStream_t st) {
  const int nvec = p.N >> 3;
  if (nvec <= 32) return launch_rows<KIND, 32, 1>(p, st);
  if (nvec <= 64) return launch_rows<KIND, 32, 2>(p, st);
  if (nvec <= 128) return launch_rows<KIND, 32, 4>(p, st);
  if (nvec <= 256) return launch_rows<KIND, 256, 1>(p, st);
  if (nvec <= 512) return launch_rows<KIND, 256, 2>(p, st);
  if (nvec <= 1024) return launch_rows<KIND, 256, 4>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_row_epilogue(int kind, const RowParams& p, cudaStream_t st) {
  switch (kind) {
    case EPI_LN: return dispatch_rows<EPI_LN>(p, st);
    case EPI_RMS_MAX: return dispatch_rows<EPI_RMS_MAX>(p, st);
    case EPI_SOFTMAX: return dispatch_rows<EPI_SOFTMAX>(p, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_wide_row_finish(int kind, const RowParams& p, const float2* partials, int nblocks, int block, cudaStream_t st) {
  const long long rows = static_cast<long long>(p.batch) * p.M;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  cfg.gridDim = dim3(static_cast<unsigned>((rows + 7) / 8), 1, 1);  // eight rows (warps) per block
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // its launch overlaps the first kernel's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic_launch_enabled() ? 1 : 0;
  count_launch();
  if (kind == EPI_LN) return cudaLaunchKernelEx(&cfg, wide_row_finish_kernel<EPI_LN>, p, partials, nblocks, block, rows);
  if (kind == EPI_RMS_MAX) return cudaLaunchKernelEx(&cfg, wide_row_finish_kernel<EPI_RMS_MAX>, p, partials, nblocks, block, rows);
  return cudaErrorInvalidValue;
}

cudaError_t launch_bias_gelu(uint16_t* P, const uint16_t* bias, long long rows, int n, cudaStream_t st) {
  const long long nvec_total = rows * (n >> 3);
  const unsigned blocks = static_cast<unsigned>((nvec_total + 255) / 256);
  count_launch();
  bias_gelu_kernel<<<blocks, 256, 0, st>>>(P, bias, nvec_total, n >> 3);
  return cudaGetLastError();
}

}  // namespace comfuse
