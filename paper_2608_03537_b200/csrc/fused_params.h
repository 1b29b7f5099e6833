// Kernel parameter block of the GEMM -> subgraph kernels (plain data, shared by host and device code).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace comfuse {

// EPI_RMS_MAX_LINEAR: the RMSNorm op list without its GELU (a kernel instantiation of its own, chosen by FusedParams::no_activation)
// EPI_ELEMENTWISE: Y = act(alpha * Acc + bias), no reduction: the plain GEMM's tiling (any N, all SMs, two accumulator
// slots) with the activation in its store epilogue; FusedParams::activation is the comfuse_op_t of the unary node (0 = none)
enum : int { EPI_NONE = 0, EPI_LN = 1, EPI_RMS_MAX = 2, EPI_SOFTMAX = 3, EPI_RMS_MAX_LINEAR = 4, EPI_PROGRAM = 5, EPI_ELEMENTWISE = 6 };

// ---------------------------------------------------------------------------------------------------------------
// Stage program: an epilogue given as data, lowered for the on-chip interpreter of the fused kernel (EPI_PROGRAM).
// The Stage-Stream model (Sec. 3) with ONE resident tensor x (the accumulator's TMEM columns) and per-row scalars:
//   pass 0:   v = entry(acc)            -> x (written back to TMEM); reductions whose input is available in pass 0
//   pass s:   for every reduction of pass s: u = chain_r(x) -> thread partial -> cluster merge -> scalar
//             then the per-row scalar instructions of that boundary
//   the pass the terminal belongs to also computes y = final(x), rounds and stores it, and accumulates the
//   reductions that take y itself as input (the chained second reduction of Sec. 3.2).
// Chains are accumulator-machine code on a 32-column fragment: v = op(v) or v = v (op) operand.
enum ChainOperand : uint8_t {
  CHO_NONE = 0,
  CHO_CONST,     // imm
  CHO_SCALAR,    // per-row scalar `index`
  CHO_ROWVEC,    // row-vector parameter staged in shared memory, `index` = 0..2
  CHO_RESIDUAL,  // the full-tensor parameter (entry chain only; delivered through the operand ring)
  CHO_MASK,      // causal mask: 0 where column <= row, -inf above the diagonal
  CHO_X,         // the resident tensor itself (the accumulator, inside the entry chain): gates such as x * sigmoid(x)
  CHO_T          // temporary fragment `index` (kernels generated for the program only): two computed tensors meet in a node
};
// chain opcodes: the comfuse_op_t values of the unary / binary nodes, plus the reversed non-commutative forms
constexpr int kChainRsub = 38;  // v = operand - v
constexpr int kChainRdiv = 39;  // v = operand / v
constexpr int kChainMov = 40;   // v = operand (a chain that starts from a broadcast: sigmoid(row vector), ...)
// micro-instructions of a pass's stream (besides the chain operations)
constexpr int kChainXsave = 66;  // x = v (pass 0, after the entry chain)
constexpr int kChainXload = 67;  // v = x
constexpr int kChainAcc = 68;    // accumulate v into the thread-local partial of reduction `index`
constexpr int kChainEmit = 69;   // round v and stage it for the output store
constexpr int kChainTsave = 70;  // temporary `index` = v (generated kernels only: the temporaries are registers there)
constexpr int kStageMaxTemps = 3;

struct ChainInstr {
  uint8_t op;
  uint8_t operand;  // ChainOperand
  int16_t index;
  float imm;
};

struct StageReduction {
  uint8_t pass;        // the pass in which its input is available
  uint8_t op;          // comfuse_op_t of the reduction (sum, mean, max, min, prod, argmax; Top-K: argmax)
  uint8_t on_terminal; // input is y itself: accumulated in the terminal's pass from the unrounded y
  uint8_t dst;         // per-row scalar it defines (unused by Top-K)
  // Top-K (the StreamReduction node's parameter K, Sec. 5): K rounds of an arg max.  Round 0 is the arg max the pass's
  // stream accumulates anyway; every further round sweeps the resident tensor again with code[code_lo .. code_hi) -- the
  // instructions that lead from x to this reduction's ACC -- and takes the best element that ranks behind the previous
  // pick (value falling, column rising).  The picks go straight to the row outputs that name this reduction.
  uint8_t k;           // 0 = an ordinary reduction
  uint8_t code_lo, code_hi;
  uint8_t pad;
};

struct ScalarInstr {   // per-row arithmetic at a stage boundary: s[dst] = op(a, b)
  uint8_t after_pass;  // runs after the merges of this pass
  uint8_t op;
  uint8_t dst;
  uint8_t a_kind, b_kind;  // CHO_CONST or CHO_SCALAR
  uint8_t a, b;
  uint8_t pad;
  float a_imm, b_imm;
};

struct StageRowOutput {
  void* ptr;        // fp32 [batch * M], int32 for an arg max; [batch * M, K] for a Top-K output
  uint8_t scalar;
  uint8_t is_int;
  uint8_t topk_red; // 1 + the Top-K reduction whose values (is_int = 0) or columns (is_int = 1) this output takes, 0 = none
  uint8_t pad[5];
};

constexpr int kStageMaxCode = 80, kStageMaxRed = 6, kStageMaxScalarInstr = 12, kStageMaxScalars = 16, kStageMaxRowOut = 6,
              kStageMaxPasses = 4, kStageMaxTopK = 8;

// The order in which the kernel takes a program's sweeps over the resident tensor: every pass, and behind a pass's merges
// the further rounds of its Top-K reductions.  Built on the host, so the kernel walks a table instead of deciding -- and
// the table is a compile-time constant when the program is compiled into the kernel.
struct SweepStep {
  uint8_t i0, i1;      // micro-instruction range code[i0 .. i1)
  int8_t topk_r;       // -1: a pass (its merges and per-row arithmetic follow); >= 0: a Top-K sweep of this reduction
  uint8_t topk_round;  // Top-K sweep: which pick it looks for (1 .. K-1; round 0 is the pass's own arg max)
  uint8_t pass;
  uint8_t release;     // the accumulator is handed back behind this step (the last one)
  uint8_t pad[2];
};
constexpr int kStageMaxSweeps = kStageMaxPasses + kStageMaxRed * (kStageMaxTopK - 1);

struct StageProgram {
  uint8_t n_red, n_scalar_instr, n_passes, terminal_pass;
  uint8_t n_row_out;
  uint8_t x_writeback;  // x goes back to tensor memory even in a one-pass program (a Top-K re-reads it)
  uint8_t uses_temps;   // the code uses temporaries (CHO_T, TSAVE): runs as generated code only, the interpreter refuses it
  uint8_t pad[1];
  // per pass, the micro-instruction stream run on every 32-column fragment: code[pass_off[s] .. pass_off[s + 1]).
  // pass 0: entry chain, XSAVE; every pass: per reduction of the pass (XLOAD if v was changed,) its chain, ACC; the
  // terminal's pass: (XLOAD,) final chain, ACC of the reductions on y, EMIT.
  uint8_t pass_off[kStageMaxPasses + 1];
  uint8_t n_sweeps;
  uint8_t pad2[2];
  SweepStep sweep[kStageMaxSweeps];
  ChainInstr code[kStageMaxCode];
  StageReduction red[kStageMaxRed];
  ScalarInstr sc[kStageMaxScalarInstr];
  StageRowOutput out[kStageMaxRowOut];
};

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
  int activation;     // EPI_ELEMENTWISE: relu / gelu_tanh / tanh / sigmoid as comfuse_op_t, 0 = none
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
  const uint16_t* mask;  // softmax kinds: additive bf16 mask [M, N] (ld = N), shared by all batches, or null
  int b_nk;              // the B operand is stored [N, K] (K-major tensor-core operand)
  int wide;
  int wide_block;   // columns per block of the two-kernel form (the instantiation that runs each block)
  float2* wide_partials;
  // Cross-CTA aggregation of the row statistics (Sec. 3.1): 0 = all-to-all (every CTA sends its partial to every peer),
  // 1 = leader-follower (partials go to column range 0, which merges and sends the result back).  Same merge order,
  // hence the same bits, either way.
  int leader_reduce;
  StageProgram program;  // EPI_PROGRAM only
  unsigned int* status;
  unsigned long long timeout_ns;
  unsigned long long* trace;  // phase timestamps of CTA 0 (builds with -DCOMFUSE_TRACE only), else null
  int trace_flags;            // tracing builds: bit 0 = skip the output stores, bit 1 = skip the UMMAs
};

// the kernels take four 128-byte tensor maps and this block by value: 4 KB of parameter space
static_assert(sizeof(FusedParams) + 4 * 128 <= 4096, "kernel parameter space");

}  // namespace comfuse
