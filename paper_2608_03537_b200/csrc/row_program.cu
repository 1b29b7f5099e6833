// Row-program kernel: evaluates a lowered epilogue program (fusion_spec.h) on the rows of a materialised GEMM result.
// This is the standard pathway for programs that do not lower to a fused instantiation (Sec. 5.2: operators outside
// the fused pattern set fall back to the standard compilation pathway).
//
// One thread block per row.  Tensor-valued computed nodes live in row-sized fp32 buffers in shared memory (slot
// numbers are assigned on the host by liveness); every thread owns the column pairs (2j, 2j+1), j = tid, tid + T, ...
// of every buffer, so element-wise instructions need no barrier between them.  A reduction is a stage boundary
// (Sec. 3): the block reduces, the per-row result goes to a small scalar table that later instructions read.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "comfuse.h"
#include "fusion_spec.h"
#include "host_common.h"

namespace comfuse {

namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__device__ __forceinline__ uint32_t float_to_bf16_rn(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u;  // NaN
  return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

__device__ __forceinline__ float unary_op(int op, float a) {
  switch (op) {
    case COMFUSE_OP_NEG: return -a;
    case COMFUSE_OP_ABS: return fabsf(a);
    case COMFUSE_OP_SQUARE: return a * a;
    case COMFUSE_OP_SQRT: return sqrtf(a);
    case COMFUSE_OP_RSQRT: return 1.f / sqrtf(a);
    case COMFUSE_OP_RECIP: return 1.f / a;
    case COMFUSE_OP_EXP: return expf(a);
    case COMFUSE_OP_LOG: return logf(a);
    case COMFUSE_OP_TANH: return tanhf(a);
    case COMFUSE_OP_RELU: return fmaxf(a, 0.f);
    case COMFUSE_OP_GELU_TANH: return 0.5f * a * (1.f + tanhf(0.7978845608028654f * (a + 0.044715f * a * a * a)));
    case COMFUSE_OP_SIGMOID: return 1.f / (1.f + expf(-a));
    default: return a;
  }
}

__device__ __forceinline__ float binary_op(int op, float a, float b) {
  switch (op) {
    case COMFUSE_OP_ADD: return a + b;
    case COMFUSE_OP_SUB: return a - b;
    case COMFUSE_OP_MUL: return a * b;
    case COMFUSE_OP_DIV: return a / b;
    case COMFUSE_OP_MAX: return fmaxf(a, b);
    case COMFUSE_OP_MIN: return fminf(a, b);
    default: return a;
  }
}

struct RowCtx {
  const RowProgram* P;
  float* slots;
  const float* scalars;
  long long row_lin;  // batch * M + row
  int row;            // row inside the batch
};

// The pair of columns (2j, 2j+1) of an operand.
__device__ __forceinline__ float2 fetch(const RowCtx& c, const Operand& o, int j) {
  const RowProgram& P = *c.P;
  switch (o.kind) {
    case OPK_SLOT: return reinterpret_cast<const float2*>(c.slots + static_cast<size_t>(o.index) * P.N)[j];
    case OPK_SCALAR: { const float v = c.scalars[o.index]; return make_float2(v, v); }
    case OPK_CONST: return make_float2(o.imm, o.imm);
    case OPK_ROWVEC: {
      const uint32_t w = reinterpret_cast<const uint32_t*>(P.params[o.index])[j];
      return make_float2(bf16_bits_to_float(w & 0xFFFFu), bf16_bits_to_float(w >> 16));
    }
    case OPK_TENSOR: {
      const uint32_t w = reinterpret_cast<const uint32_t*>(P.params[o.index] + c.row_lin * P.param_ld[o.index])[j];
      return make_float2(bf16_bits_to_float(w & 0xFFFFu), bf16_bits_to_float(w >> 16));
    }
    case OPK_ACC: {
      const uint32_t w = reinterpret_cast<const uint32_t*>(P.Z + c.row_lin * P.N)[j];
      return make_float2(bf16_bits_to_float(w & 0xFFFFu), bf16_bits_to_float(w >> 16));
    }
    case OPK_MASK: return make_float2(2 * j <= c.row ? 0.f : -CUDART_INF_F, 2 * j + 1 <= c.row ? 0.f : -CUDART_INF_F);
    default: return make_float2(0.f, 0.f);
  }
}

__device__ __forceinline__ float scalar_of(const RowCtx& c, const Operand& o) {
  return o.kind == OPK_SCALAR ? c.scalars[o.index] : o.imm;
}

// (value, column) pairs of the arg max: the larger value wins, equal values keep the lower column
__device__ __forceinline__ void argmax_merge(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

__global__ void __launch_bounds__(256) row_program_kernel(const __grid_constant__ RowProgram P) {
  extern __shared__ __align__(16) float s_slots[];
  __shared__ float s_scalar[kRowMaxScalars];
  __shared__ float s_red[8];
  __shared__ int s_redi[8];

  const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, wid = tid >> 5, nwarps = T >> 5;
  const long long row_lin = blockIdx.x;
  RowCtx c;
  c.P = &P;
  c.slots = s_slots;
  c.scalars = s_scalar;
  c.row_lin = row_lin;
  c.row = static_cast<int>(row_lin % P.M);
  const int pairs = P.N >> 1;

  for (int k = 0; k < P.n_instr; ++k) {
    const RowInstr& in = P.ins[k];
    const int op = in.op;
    if (op == COMFUSE_OP_RED_TOPK_VALUES || op == COMFUSE_OP_RED_TOPK_INDICES) {
      // ---- Top-K: K rounds of a block arg max over the elements that rank after the previous pick in the order
      // (value falling, column rising); round r's pick goes straight to the row output
      const int K = in.b.index;
      float last_v = CUDART_INF_F;
      int last_i = -1;
      for (int r = 0; r < K; ++r) {
        float acc = -CUDART_INF_F;
        int idx = 0x7FFFFFFF;
        for (int j = tid; j < pairs; j += T) {
          const float2 v = fetch(c, in.a, j);
          const float e[2] = {v.x, v.y};
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int col = 2 * j + u;
            const bool eligible = e[u] < last_v || (e[u] == last_v && col > last_i);
            if (eligible && (e[u] > acc || (e[u] == acc && col < idx))) { acc = e[u]; idx = col; }
          }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) argmax_merge(acc, idx, __shfl_xor_sync(0xFFFFFFFFu, acc, off), __shfl_xor_sync(0xFFFFFFFFu, idx, off));
        if (lane == 0) { s_red[wid] = acc; s_redi[wid] = idx; }
        __syncthreads();
        float rv = s_red[0];
        int ri = s_redi[0];
        for (int w = 1; w < nwarps; ++w) argmax_merge(rv, ri, s_red[w], s_redi[w]);
        __syncthreads();  // everyone has read the partials before the next round overwrites them
        last_v = rv;
        last_i = ri;
        if (tid == 0 && in.dst >= 0) {
          if (op == COMFUSE_OP_RED_TOPK_INDICES) static_cast<int*>(P.row_out[in.dst])[row_lin * K + r] = ri;
          else static_cast<float*>(P.row_out[in.dst])[row_lin * K + r] = rv;
        }
      }
    } else if (op >= COMFUSE_OP_RED_SUM) {
      // ---- stage boundary: block-wide reduction of operand a over the row
      const bool is_max = op == COMFUSE_OP_RED_MAX || op == COMFUSE_OP_RED_ARGMAX;
      float acc = op == COMFUSE_OP_RED_PROD ? 1.f : is_max ? -CUDART_INF_F : op == COMFUSE_OP_RED_MIN ? CUDART_INF_F : 0.f;
      int idx = 0x7FFFFFFF;
      for (int j = tid; j < pairs; j += T) {
        const float2 v = fetch(c, in.a, j);
        switch (op) {
          case COMFUSE_OP_RED_SUM:
          case COMFUSE_OP_RED_MEAN: acc += v.x + v.y; break;
          case COMFUSE_OP_RED_MAX: acc = fmaxf(acc, fmaxf(v.x, v.y)); break;
          case COMFUSE_OP_RED_MIN: acc = fminf(acc, fminf(v.x, v.y)); break;
          case COMFUSE_OP_RED_PROD: acc *= v.x * v.y; break;
          default:  // arg max; columns rise with j, so a strict compare keeps the lowest column
            if (v.x > acc) { acc = v.x; idx = 2 * j; }
            if (v.y > acc) { acc = v.y; idx = 2 * j + 1; }
            break;
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xFFFFFFFFu, acc, off);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, idx, off);
        switch (op) {
          case COMFUSE_OP_RED_SUM:
          case COMFUSE_OP_RED_MEAN: acc += o; break;
          case COMFUSE_OP_RED_MAX: acc = fmaxf(acc, o); break;
          case COMFUSE_OP_RED_MIN: acc = fminf(acc, o); break;
          case COMFUSE_OP_RED_PROD: acc *= o; break;
          default: argmax_merge(acc, idx, o, oi); break;
        }
      }
      if (lane == 0) { s_red[wid] = acc; s_redi[wid] = idx; }
      __syncthreads();
      if (tid == 0) {
        float r = s_red[0];
        int ri = s_redi[0];
        for (int w = 1; w < nwarps; ++w) {
          const float o = s_red[w];
          switch (op) {
            case COMFUSE_OP_RED_SUM:
            case COMFUSE_OP_RED_MEAN: r += o; break;
            case COMFUSE_OP_RED_MAX: r = fmaxf(r, o); break;
            case COMFUSE_OP_RED_MIN: r = fminf(r, o); break;
            case COMFUSE_OP_RED_PROD: r *= o; break;
            default: argmax_merge(r, ri, o, s_redi[w]); break;
          }
        }
        if (op == COMFUSE_OP_RED_MEAN) r /= static_cast<float>(P.N);
        if (op == COMFUSE_OP_RED_ARGMAX) r = static_cast<float>(ri);
        s_scalar[in.dst] = r;
      }
      __syncthreads();
    } else if (in.dst_scalar) {
      // ---- arithmetic on per-row values (e.g. rsqrt(var + eps)): one thread, then everyone may read it
      if (tid == 0) {
        const float a = scalar_of(c, in.a);
        s_scalar[in.dst] = op >= COMFUSE_OP_ADD ? binary_op(op, a, scalar_of(c, in.b)) : unary_op(op, a);
      }
      __syncthreads();
    } else {
      // ---- element-wise node over this thread's column pairs
      float2* dst = reinterpret_cast<float2*>(s_slots + static_cast<size_t>(in.dst) * P.N);
      if (op >= COMFUSE_OP_ADD) {
        for (int j = tid; j < pairs; j += T) {
          const float2 a = fetch(c, in.a, j), b = fetch(c, in.b, j);
          dst[j] = make_float2(binary_op(op, a.x, b.x), binary_op(op, a.y, b.y));
        }
      } else {
        for (int j = tid; j < pairs; j += T) {
          const float2 a = fetch(c, in.a, j);
          dst[j] = make_float2(unary_op(op, a.x), unary_op(op, a.y));
        }
      }
    }
  }

  // ---- terminal node: round once, store
  const int b = static_cast<int>(row_lin / P.M);
  uint32_t* y = reinterpret_cast<uint32_t*>(P.Y + static_cast<long long>(b) * P.batch_stride_y + static_cast<long long>(c.row) * P.ldy);
  for (int j = tid; j < pairs; j += T) {
    const float2 v = fetch(c, P.terminal, j);
    y[j] = float_to_bf16_rn(v.x) | (float_to_bf16_rn(v.y) << 16);
  }
  if (tid == 0) {
    for (int r = 0; r < P.n_row_out; ++r) {
      if (P.row_out_src[r].kind == OPK_NONE) continue;  // a Top-K node: already written
      const float v = scalar_of(c, P.row_out_src[r]);
      if (P.row_out_int[r]) static_cast<int*>(P.row_out[r])[row_lin] = static_cast<int>(v);
      else static_cast<float*>(P.row_out[r])[row_lin] = v;
    }
  }
}

}  // namespace

cudaError_t launch_row_program(const RowProgram& prog, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(prog.n_slots) * prog.N * sizeof(float);
  if (smem > kRowMaxSlotBytes) return cudaErrorInvalidValue;
  // the shared-memory opt-in is a per-device attribute of the kernel
  constexpr int kMaxDev = 64;
  static bool attr_set[kMaxDev] = {};
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;
  if (!attr_set[di] || dev->device >= kMaxDev) {
    cudaError_t e = cudaFuncSetAttribute(row_program_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kRowMaxSlotBytes));
    if (e != cudaSuccess) return e;
    attr_set[di] = true;
  }
  const int threads = prog.N >= 1024 ? 256 : prog.N >= 256 ? 128 : 64;
  const long long rows = static_cast<long long>(prog.batch) * prog.M;
  row_program_kernel<<<static_cast<unsigned>(rows), threads, smem, st>>>(prog);
  count_launch();
  return cudaGetLastError();
}

}  // namespace comfuse
