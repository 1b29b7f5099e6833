// Lowered form of an epilogue program (Sec. 5.2 Fusion Spec IR -> Sec. 5.4 backend mapping): what the row-program
// kernel executes, and what the host-side analysis records about a program.  Plain data.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace comfuse {

// Where an instruction reads a value from.
enum OperandKind : uint8_t {
  OPK_NONE = 0,
  OPK_SLOT,    // row-sized fp32 buffer `index` in shared memory (a computed tensor-valued node)
  OPK_SCALAR,  // per-row value `index` (a reduction result, or arithmetic on such values)
  OPK_CONST,   // `imm`
  OPK_ROWVEC,  // parameter `index`, bf16 [N]
  OPK_TENSOR,  // parameter `index`, bf16 [batch, M, N]
  OPK_ACC,     // the GEMM result (bf16 Z in the workspace)
  OPK_MASK     // causal mask: 0 where column <= row, -inf above the diagonal
};

struct Operand {
  uint8_t kind;
  uint8_t pad;
  int16_t index;
  float imm;
};

// One computed node: dst = op(a, b).  dst is a shared-memory slot, or a per-row scalar when `dst_scalar` is set
// (reductions and arithmetic on per-row values).
struct RowInstr {
  uint8_t op;  // comfuse_op_t value (all are below 256)
  uint8_t dst_scalar;
  int16_t dst;
  Operand a, b;
};

constexpr int kRowMaxInstr = 128;
constexpr int kRowMaxParams = 12;
constexpr int kRowMaxRowOut = 8;
constexpr int kRowMaxScalars = 128;
constexpr size_t kRowMaxSlotBytes = 200 * 1024;  // shared memory the row buffers may take

struct RowProgram {
  int batch, M, N;
  int n_instr, n_slots, n_row_out;
  const uint16_t* Z;  // [batch, M, N] bf16, dense
  uint16_t* Y;
  long long ldy, batch_stride_y;
  Operand terminal;
  const uint16_t* params[kRowMaxParams];
  long long param_ld[kRowMaxParams];
  void* row_out[kRowMaxRowOut];
  Operand row_out_src[kRowMaxRowOut];
  uint8_t row_out_int[kRowMaxRowOut];
  RowInstr ins[kRowMaxInstr];
};
static_assert(sizeof(RowProgram) <= 4000, "passed by value as a kernel parameter");

cudaError_t launch_row_program(const RowProgram& prog, cudaStream_t st);

}  // namespace comfuse
