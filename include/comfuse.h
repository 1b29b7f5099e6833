/*
 * comfuse.h -- C ABI of the B200 (sm_100a) joint compute-memory fusion library.
 *
 * One bf16 tensor-core GEMM (or a back-to-back pair of GEMMs) whose fp32 result is consumed on-chip by
 * an elementwise/reduction subgraph, without writing the GEMM result to global memory (ComFuse: Sec. 1 states
 * the problem of fusing the compute-bound operator with its memory-bound consumers; Sec. 3 gives the staged
 * execution model of the epilogue; Sec. 4 the back-to-back GEMM).
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers unless stated otherwise; the caller owns every buffer.
 *     The library allocates no device memory; its only device state is a small status word that lives
 *     in the loaded module.  (A kernel generated at run time for an epilogue program -- comfuse_gemm_spec, below -- is a
 *     module of its own, loaded by the first launch that needs it.)
 *   - Tensors are row-major bf16 (2 bytes/element); leading dimensions are in ELEMENTS.
 *     Pointers must be 16-byte aligned and leading dimensions / batch strides multiples of 8 elements.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     return without synchronising.  Arguments are validated before anything is launched; a non-OK
 *     return means nothing was enqueued.
 *   - Device-side waits are bounded.  A wait that expires makes the kernel finish early and records
 *     COMFUSE_ERR_TIMEOUT in the status word, read with comfuse_last_device_status().
 *   - `fused = 1` selects the single fused kernel; `fused = 0` selects the in-library unfused path with
 *     identical semantics (GEMM kernel writes a bf16 intermediate to `workspace`, a row kernel finishes).
 *   - No C++ exceptions cross this boundary.  The library needs compute capability 10.x.
 */
#ifndef COMFUSE_H_
#define COMFUSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COMFUSE_OK = 0,
  COMFUSE_ERR_INVALID_ARG = 1,  /* NULL where a pointer is required, non-positive size, bad enum        */
  COMFUSE_ERR_UNSUPPORTED = 2,  /* shape / op list has no compiled fused instantiation (try fused = 0)    */
  COMFUSE_ERR_ALIGNMENT = 3,    /* pointer not 16-byte aligned or leading dimension not a multiple of 8  */
  COMFUSE_ERR_WORKSPACE = 4,    /* workspace NULL or smaller than comfuse_*_workspace_size() reports      */
  COMFUSE_ERR_ARCH = 5,         /* current device is not compute capability 10.x                           */
  COMFUSE_ERR_CUDA = 6,         /* a CUDA runtime / driver call failed (launch, tensor-map encode, ...)   */
  COMFUSE_ERR_TIMEOUT = 7,      /* a bounded device-side wait expired (reported by last_device_status)    */
  COMFUSE_ERR_BOUNDS = 8        /* checked build only (-DCOMFUSE_CHECKED): a bounds predicate inside a kernel failed;
                                   the access was skipped (reported by last_device_status)                 */
} comfuse_status_t;

/* The memory-intensive subgraph fused behind the GEMM, as a fixed, topologically ordered op list
 * (Sec. 5.2: the Fusion Spec IR is an ordered node list plus a table of runtime parameters; here the
 * list is chosen by enum and the parameter table is comfuse_epilogue_args_t).  Reductions are over the
 * last dimension N and are the stage boundaries of Sec. 3. */
typedef enum {
  /* Y = LayerNorm(alpha*A.B + bias + R) * gamma + beta  -- Sec. 3.2 / Fig. 3 (x = alpha*Acc + Bias; mean; x - mean) */
  COMFUSE_EPI_BIAS_RES_LAYERNORM = 0,
  /* H = GELU_tanh(alpha*A.B + bias) + R;  Y = H * rsqrt(mean(H^2) + eps) * gamma;  then a second, chained
   * reduction: row_max[i] = max_j Y, row_argmax[i] = lowest such j  -- Sec. 2.2 (MatMul + RMSNorm), Sec. 3.2 */
  COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX = 1,
  /* P = softmax(alpha*A.B + mask) over the last dim  -- Sec. 5 (ReduceMode softmax), Sec. 6.1 (attention scores) */
  COMFUSE_EPI_SCALE_MASK_SOFTMAX = 2,
  /* Y = act(alpha*A.B + bias), act in {none, ReLU, GELU_tanh, tanh, sigmoid}: a reduction-free epilogue (any N that is a
   * multiple of 8, the plain GEMM's tiling).  Reported by comfuse_spec_plan for programs that lower to it and run by
   * comfuse_gemm_spec; comfuse_gemm_epilogue does not take this kind (INVALID_ARG). */
  COMFUSE_EPI_BIAS_ACTIVATION = 3
} comfuse_epilogue_kind_t;

typedef enum {
  COMFUSE_MASK_NONE = 0,
  COMFUSE_MASK_CAUSAL = 1,   /* 0 where column <= row, -inf elsewhere; requires M == N            */
  COMFUSE_MASK_ADDITIVE = 2  /* bf16 [M, N] tensor (ld = N) added to the scaled (and soft-capped) scores,
                                shared by all batches; may hold -inf: such entries give exact zeros, a
                                row with nothing else gives a row of zeros                        */
} comfuse_mask_t;

typedef struct {
  int32_t batch;            /* >= 1; A, B, R, Y, row_max, row_argmax are batched, vectors are shared   */
  int32_t M, N, K;          /* A is [M, K], B is [K, N] (N contiguous), Y and R are [M, N]              */
  int64_t lda, ldb, ldr, ldy;
  int64_t batch_stride_a, batch_stride_b, batch_stride_r, batch_stride_y;   /* elements */
  int32_t kind;             /* comfuse_epilogue_kind_t */
  int32_t mask;             /* comfuse_mask_t, SOFTMAX kind only */
  float alpha;              /* scales the accumulator before anything else */
  float eps;                /* added to the variance / mean square inside the square root */
  int32_t fused;            /* 1 = fused kernel, 0 = in-library unfused path */
  uint32_t flags;           /* COMFUSE_FLAG_* bits, 0 for the op lists exactly as described at the enum */
  float softcap;            /* SOFTMAX kind: if > 0, the scaled scores become softcap * tanh(alpha*A.B / softcap) before
                               the mask is added (Sec. 6.1, MatMul-Scale-TanhSoftcap-Softmax); must be 0 for other kinds */
  int32_t reserved;         /* must be 0 */
} comfuse_gemm_desc_t;

/* Variants of the op lists (the three evaluation patterns of Sec. 6.1 are LAYERNORM + POST_RELU, RMSNORM_MAX +
 * NO_ACTIVATION without a residual, and SOFTMAX with softcap > 0). */
#define COMFUSE_FLAG_POST_RELU 1u      /* BIAS_RES_LAYERNORM kind only: Y = max(Y, 0) after the affine step            */
#define COMFUSE_FLAG_NO_ACTIVATION 2u  /* BIAS_GELU_RES_RMSNORM_MAX kind only: H = alpha*A.B + bias + R, no GELU       */
/* The second operand is stored [batch, N, K] (ldb >= K: the contraction dimension contiguous, one column of the product per
 * row -- a linear layer's weight [out, in], attention keys as a layer holds them), i.e. the call computes alpha * A.B^T of
 * the stored tensors.  Every GEMM kernel of the library reads it in place as a K-major tensor-core operand (fused and
 * unfused, all kinds, same results bit for bit as with the transposed operand); the host-buffer and workspace-free entry
 * points take it too, the node-list entry point through comfuse_gemm_shape_t.flags. */
#define COMFUSE_FLAG_B_ROW_MAJOR_NK 4u

/* Runtime-parameter table of the op list.  bias, gamma, beta: bf16 device vectors of length N, shared by all batches;
 * residual: bf16 [batch, M, N] with leading dimension desc->ldr; mask: see comfuse_mask_t.  NULL means absent (bias,
 * residual: 0; gamma: 1; beta: 0).  row_max (fp32) / row_argmax (int32): [batch*M] outputs of the RMSNORM_MAX kind,
 * required there and ignored elsewhere. */
typedef struct {
  const void* bias;
  const void* residual;
  const void* gamma;
  const void* beta;
  const void* mask;
  float* row_max;
  int32_t* row_argmax;
} comfuse_epilogue_args_t;

/* Bytes of caller-provided workspace the described call can use.  Most fused calls need none.  Three cases of the LayerNorm /
 * RMSNorm kinds run as TWO kernels and report batch * M * (N / block) * 8 bytes: the fused kernel finishes stage 1 per
 * column block, stores the un-normalised row in Y as fp16 (11 significant bits) and one partial statistic per row and
 * block in the workspace; a second kernel merges the partials and rescales the row in place to bf16.
 *   - Rows wider than the largest cluster can hold on-chip (4096 < N <= 65536): the un-normalised values are materialised
 *     because they no longer fit (Sec. 2.2).  block = 256 behind a long contraction (K >= 1024, N a multiple of 256),
 *     otherwise block = 4096 (N a multiple of 4096).  The workspace is required.
 *   - Rows of 2048 .. 4096 columns (a multiple of 256) behind a long contraction (K >= 1024), block = 256: measured faster
 *     than keeping the row on chip, because the 8- and 16-CTA clusters that hold such rows leave SMs idle and cannot
 *     overlap a tile's epilogue with the next MainLoop.  Here the workspace is optional where the row length has an
 *     on-chip instantiation (2048, 4096): a call that brings none keeps the row on chip.  The same holds for rows of 512 ..
 *     1024 columns when there are so few rows that the on-chip clusters would leave most of the machine idle (fewer than about
 *     6000 rows; K >= 1536 for the LayerNorm kind, K >= 1024 for the RMSNorm kind).
 *   - Row lengths without an on-chip instantiation (the on-chip ones: 256, 512, 768, 1024, 2048, 4096 and row lengths up to
 *     a quarter shorter than one of these, which run on it with the surplus columns masked; behind contractions short
 *     enough for it to pay also 1280, 1536, 1792: ask this function) that are not a
 *     multiple of 4096 -- 1000, 1280, 1536, 1600, 3072, 5120, ... any multiple of 8 up to 65536 -- at any K, block = 256,
 *     (N + 255) / 256 blocks: the last tile may be a partial one.  The workspace is required.
 *   With these every row length that is a multiple of 8 (up to 65536 columns) has a fused form for all three kinds.
 * The results of both forms meet the same tolerances as the one-kernel path. */
comfuse_status_t comfuse_workspace_size(const comfuse_gemm_desc_t* desc, size_t* bytes);

/* GEMM -> subgraph (Sec. 3).  A, B inputs; Y output [batch, M, N] bf16, rounded once, at the store. */
comfuse_status_t comfuse_gemm_epilogue(const comfuse_gemm_desc_t* desc, const void* A, const void* B, void* Y,
                                       const comfuse_epilogue_args_t* args, void* workspace,
                                       size_t workspace_bytes, void* cuda_stream);

/* GEMM -> subgraph through the UNFUSED path without a caller workspace.  (The paper has no counterpart of this
 * entry point: it exists for callers of this library, not for the method.)
 *
 * Some callers cannot provide the workspace that comfuse_gemm_epilogue(fused = 0) needs, because they cannot
 * allocate device memory where the call happens: code in a latency-critical loop where cudaMalloc (which
 * synchronises the device) is not allowed, plug-ins that receive tensors from
 * a host framework but have no access to its allocator, or processes whose device memory is handed out entirely by
 * another component.  For them the intermediate bf16 GEMM result is kept in a fixed array of
 * COMFUSE_STATIC_SCRATCH_BYTES that is part of the library's device image; every GPU on which the library is loaded
 * holds that array until the process exits.
 *
 * Semantics are those of comfuse_gemm_epilogue with desc->fused forced to 0; desc->fused is ignored.
 *   - The call allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.
 *   - batch * M * N * 2 bytes must fit in COMFUSE_STATIC_SCRATCH_BYTES; a larger problem is rejected with
 *     COMFUSE_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address and configures the kernels it launches;
 *     that first call should come before any stream capture.  The cached address does not survive cudaDeviceReset.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it.  Nothing in it
 *     needs clearing (each call overwrites the region it later reads), but two calls whose kernels can overlap on
 *     the GPU -- different streams without an ordering between them -- race on it.  Order such calls on one stream
 *     or with events. */
#define COMFUSE_STATIC_SCRATCH_BYTES (16u << 20)
comfuse_status_t comfuse_gemm_epilogue_static_scratch(const comfuse_gemm_desc_t* desc, const void* A, const void* B,
                                                      void* Y, const comfuse_epilogue_args_t* args, void* cuda_stream);

/* Back-to-back GEMM (Sec. 4, Eq. 2) with F = GELU_tanh(. + b1) and the tail
 *   O = LayerNorm(S.W2 + b2 + X) * gamma + beta,   S = F(X.W1),
 * X [M, K], W1 [K, N1], W2 [N1, N2], all dense row-major bf16, N2 == K.  In the fused path S (and P) never
 * leave the chip: S is rounded to bf16 as the second GEMM's tensor-core operand.  Fused: K = N2 = 128, N1 a multiple of
 * 8 up to 4096 (the hidden layer streams through in chunks of 128 columns; a partial last chunk is filled with zeros,
 * which GELU keeps); other shapes: fused = 0. */
typedef enum {
  COMFUSE_B2B_MLP_GELU_LAYERNORM = 0, /* as above                                                                   */
  /* Attention form (Sec. 4, Eq. 2 with a row reduction as F; the Target-Attention workload of Sec. 6.2):
   *   O = softmax(alpha * X.W1) . W2   per batch,  softmax over the N1 source positions,
   * X [batch, M, K] queries, W1 [batch, K, N1] keys (already transposed) -- or, with COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR,
   * W1 [batch, N1, K], one key per row as an attention layer produces them --, W2 [batch, N1, N2] values, O [batch, M, N2],
   * all dense.  b1, b2, gamma, beta must be NULL, alpha > 0.  Fused: K = N2 = 128 and N1 <= 512, a multiple of 8: up to
   * 256 source positions a whole score row fits the accumulators of one CTA pair, above that it is two sub-tiles of 256
   * source positions, each exponentiated against its own row maximum, combined when O is normalised; positions from N1 up
   * to the end of the last sub-tile are loaded as zeros and take no part in the softmax.  The probabilities are rounded
   * to bf16 as the second GEMM's operand. */
  COMFUSE_B2B_SOFTMAX_ATTENTION = 1,
  /* Two-layer ReLU MLP (Sec. 4, Eq. 2 with F = ReLU(. + b1); the DLRM workload of Sec. 6.2, 1024 -> 512 -> 128):
   *   O = ReLU(ReLU(X.W1 + b1).W2 + b2),
   * X [M, K], W1 [K, N1], W2 [N1, N2]; K and N2 independent, batch = 1, gamma and beta must be NULL, b1 / b2 may be NULL.
   * Fused: N2 = 128, N1 <= 512 (a multiple of 8), any K (a multiple of 8) streamed through the first GEMM; the hidden layer is rounded
   * to bf16 as the second GEMM's operand and never leaves the chip.  Unfused: any shape, the bf16 hidden layer [M, N1] in
   * the workspace. */
  COMFUSE_B2B_MLP_RELU = 2
} comfuse_b2b_kind_t;

typedef struct {
  int32_t M, K, N1, N2;
  float eps;
  int32_t fused;
  int32_t kind;   /* comfuse_b2b_kind_t */
  int32_t batch;  /* >= 1; must be 1 for the MLP kind (its weights are shared by all rows) */
  float alpha;    /* attention kind: scale of the scores; ignored by the MLP kind */
  int32_t flags;  /* COMFUSE_B2B_FLAG_*; 0 otherwise (any other bit: COMFUSE_ERR_INVALID_ARG) */
} comfuse_b2b_desc_t;

/* Attention kind only: W1 is stored [batch, N1, K] (keys row-major, the contraction dimension contiguous).  The fused kernel
 * and the unfused path's GEMM read it in place as a K-major tensor-core operand. */
#define COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR 1

comfuse_status_t comfuse_b2b_workspace_size(const comfuse_b2b_desc_t* desc, size_t* bytes);

comfuse_status_t comfuse_b2b_gemm(const comfuse_b2b_desc_t* desc, const void* X, const void* W1, const void* b1,
                                  const void* W2, const void* b2, const void* gamma, const void* beta, void* O,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Host-buffer forms (the paper has no counterpart: it measures kernels on resident tensors).  The per-step tensors
 * selected by `host_mask` are HOST pointers (pinned memory if the copies are to be asynchronous); everything else stays a
 * device pointer as above.  The call enqueues, on `cuda_stream`: one host -> device copy per selected input into
 * `staging` (DEVICE memory owned by the caller, at least comfuse_host_staging_size() bytes, 16-byte aligned), the same
 * kernels as comfuse_gemm_epilogue, and, if COMFUSE_HOST_Y is set, one device -> host copy of the result.  Each copy moves
 * the tensor's whole strided extent ((batch-1)*batch_stride + (rows-1)*ld + cols elements), pad columns included.  Nothing
 * is allocated and nothing synchronises; the host buffers must stay valid until the stream has passed the call.
 * With one batch, A and Y in host memory, a LayerNorm / RMSNorm kind and at least 8 MB of activations the call runs as a
 * pipeline of up to eight row ranges of at least 4 MB each (rows are independent): range c is copied in on a library-owned copy stream while range c-1
 * computes on `cuda_stream` and range c-2's result is copied out on a second library-owned stream.  `cuda_stream` forks
 * into the two helper streams at the start of the call and joins them at its end, so work enqueued on it afterwards (an
 * event, the next call) is ordered behind the whole call; results are bit for bit those of the unpipelined form.  The
 * helper streams and events are created once per device at first use (COMFUSE_HOST_PIPELINE=0 disables the pipeline,
 * COMFUSE_HOST_CHUNKS=<2..32> sets the most ranges, default 8);
 * they serve one call at a time, so host threads that call these forms on the same device take turns enqueueing.
 * Errors: as comfuse_gemm_epilogue; COMFUSE_ERR_WORKSPACE also when `staging` is NULL or too small.  The description,
 * the workspace and the staging size are checked before anything is enqueued; an error that a CUDA call reports later
 * (COMFUSE_ERR_CUDA) can leave copies of this call on the stream, always joined back into `cuda_stream`'s order. */
#define COMFUSE_HOST_A 1u
#define COMFUSE_HOST_B 2u
#define COMFUSE_HOST_RESIDUAL 4u /* args->residual is a host pointer */
#define COMFUSE_HOST_Y 8u
comfuse_status_t comfuse_host_staging_size(const comfuse_gemm_desc_t* desc, uint32_t host_mask, size_t* bytes);
comfuse_status_t comfuse_gemm_epilogue_host(const comfuse_gemm_desc_t* desc, const void* A, const void* B, void* Y,
                                            const comfuse_epilogue_args_t* args, uint32_t host_mask, void* staging,
                                            size_t staging_bytes, void* workspace, size_t workspace_bytes, void* cuda_stream);
/* The same for the back-to-back GEMM: X and O are host pointers (dense), the weights and vectors device pointers; for
 * the attention kind W1 (keys) and W2 (values) are per-step tensors too and are host pointers as well. */
comfuse_status_t comfuse_b2b_host_staging_size(const comfuse_b2b_desc_t* desc, size_t* bytes);
comfuse_status_t comfuse_b2b_gemm_host(const comfuse_b2b_desc_t* desc, const void* X, const void* W1, const void* b1,
                                       const void* W2, const void* b2, const void* gamma, const void* beta, void* O,
                                       void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the device status word of the current device:
 * COMFUSE_OK, COMFUSE_ERR_TIMEOUT, COMFUSE_ERR_BOUNDS (checked build only), or COMFUSE_ERR_CUDA if the stream reports an
 * error. */
comfuse_status_t comfuse_last_device_status(void* cuda_stream);

/* Number of kernels this library has launched in this process since it was loaded (for accounting). */
uint64_t comfuse_launch_count(void);

/* Failure-detection self-test (the paper has no counterpart).  Launches one small kernel whose threads wait on a barrier
 * that nothing signals, with a limit of `timeout_ms` (1..1000).  The waits must expire: the kernel ends normally, the
 * device status word then reads COMFUSE_ERR_TIMEOUT (see comfuse_last_device_status) and the CUDA context stays usable.
 * If `expired_waits` (a HOST pointer) is not NULL the call synchronises the stream and stores how many threads saw an
 * expired or aborted wait (all 64). */
comfuse_status_t comfuse_selftest_bounded_wait(uint32_t timeout_ms, void* cuda_stream, uint32_t* expired_waits);

/* Checked-build self-test (the paper has no counterpart).  Launches one small kernel that evaluates a bounds predicate
 * which is false, in front of an access it therefore skips.  In a library built with -DCOMFUSE_CHECKED the device status
 * word then reads COMFUSE_ERR_BOUNDS; in the ordinary build the predicates are compiled out, the kernel does nothing and
 * the status stays COMFUSE_OK.  `*checked_build` (a HOST pointer, may be NULL) receives 1 or 0 accordingly.  Nothing is
 * read or written out of bounds in either build. */
comfuse_status_t comfuse_selftest_bounds_predicate(void* cuda_stream, int32_t* checked_build);

const char* comfuse_status_string(comfuse_status_t status);

/* ------------------------------------------------------------------------------------------------------------
 * Epilogue given as DATA (Sec. 5.2 Fusion Spec IR, Sec. 5.3 reduction subgraph splitting, Sec. 5.4 backend mapping).
 *
 * The memory-intensive subgraph is a topologically ordered list of nodes of four categories -- accumulator entry,
 * broadcast, element-wise computation, reduction over the last dimension N -- with edges to EARLIER nodes, one
 * terminal node (its value is stored to Y as bf16, rounded once) and a table of runtime parameters.  A reduction
 * yields one value per row that later element-wise nodes may use (broadcast along the row); that is how LayerNorm,
 * RMSNorm and Softmax are spelled with primitive nodes.  All arithmetic is fp32.
 *
 * What the library does with a program (the two mappings of Sec. 5):
 *   1. checks it (closure: a node outside this vocabulary, a forward edge, a mistyped parameter is rejected with
 *      COMFUSE_ERR_INVALID_ARG, nothing is dropped silently), types every node (tensor / per-row / constant) and
 *      splits it into stages at the reduction nodes: stage(node) = max over its inputs of stage(input), plus one
 *      behind a reduction;
 *   2. lowers it: a program whose stages have the shape of a compiled fused instantiation (affine entry
 *      [activation] [+ residual] -> LayerNorm | RMSNorm [-> max/argmax] | softmax, or a reduction-free act(alpha*acc + bias),
 *      in any spelling the canonicaliser recognises: operand order of commutative nodes, optional nodes absent) runs as
 *      that ONE fused kernel
 *      (path COMFUSE_SPEC_PATH_FUSED_KERNEL); a program in which ONE tensor can stay resident across the reductions --
 *      the accumulator or something computed from it before the first reduction -- and every other tensor-valued
 *      expression can be recomputed from it, from constants, per-row values, row vectors, the causal mask and (in the
 *      first pass only) one full tensor, runs as ONE fused kernel whose epilogue executes the stages over the on-chip
 *      accumulator (COMFUSE_SPEC_PATH_FUSED_PROGRAM; N in {256, 512, 768, 1024, 2048, 4096}; at most 3 row vectors, 6
 *      reductions, 6 row outputs, 4 passes, 80 micro-instructions; the reductions sum, mean, max, min, prod, argmax merge
 *      across the cluster).  Expressions in which two COMPUTED tensors meet (relu(x) * tanh(x)) need temporaries, which
 *      exist in the generated form of the kernel only (3. below): the interpreter (`fused` = 2) sends such a program to the
 *      row program; the generated form also exists at N in {1280, 1536, 1792, 2560, 3072, 3584}; any other valid program runs on the standard pathway
 *      (COMFUSE_SPEC_PATH_ROW_PROGRAM): the GEMM kernel writes bf16 Z to the workspace and one row-program kernel
 *      evaluates the node list per row with the row resident in shared memory, one pass per stage.
 *   3. on request (`fused` = 3) GENERATES the fused kernel for the program (Sec. 5: the fused epilogue as generated code):
 *      the FUSED_PROGRAM kernel is compiled at run time with the program's structure as a compile-time table, so that the
 *      interpreter's loops unroll and its dispatches fold into straight-line code; same lowering, same limits, same
 *      merge order.  Results equal the interpreter's except where the compiler contracts a multiply and the addition of
 *      the next node into one fused multiply-add (one rounding instead of two); with COMFUSE_GENERATED_FMAD=0 in the
 *      environment kernels are compiled without contraction and the results are bit-identical.  Constants (CONST nodes) and pointers stay run-time
 *      arguments: programs that differ only in those share a kernel.  The first call that needs a kernel compiles it
 *      (NVRTC from the CUDA toolkit, one to three seconds, on the calling thread) and keeps it for the life of the process;
 *      make that call, or comfuse_gemm_spec_prepare, before any stream capture.  With COMFUSE_KERNEL_CACHE=<directory>
 *      in the environment the device images are also kept on disk, and a later process loads them instead of compiling.  Where the compiler is available `fused` = 1
 *      takes this form too whenever it would otherwise interpret (COMFUSE_GENERATE=0 in the environment keeps the
 *      interpreter); comfuse_spec_plan reports COMFUSE_SPEC_PATH_FUSED_PROGRAM for both, they are the same lowering.
 */
typedef enum {
  COMFUSE_OP_ACC = 0,          /* accumulator entry: (A.B)[i, j]                                      */
  COMFUSE_OP_CONST = 1,        /* scalar broadcast of `imm`                                           */
  COMFUSE_OP_ROWVEC = 2,       /* row-vector broadcast: params[param][j], bf16 [N]                    */
  COMFUSE_OP_TENSOR = 3,       /* full tensor: params[param][i, j], bf16 [batch, M, N], ld = param_ld */
  COMFUSE_OP_CAUSAL_MASK = 4,  /* 0 where j <= i, -inf above the diagonal                             */
  COMFUSE_OP_NEG = 16, COMFUSE_OP_ABS = 17, COMFUSE_OP_SQUARE = 18, COMFUSE_OP_SQRT = 19, COMFUSE_OP_RSQRT = 20,
  COMFUSE_OP_RECIP = 21, COMFUSE_OP_EXP = 22, COMFUSE_OP_LOG = 23, COMFUSE_OP_TANH = 24, COMFUSE_OP_RELU = 25,
  COMFUSE_OP_GELU_TANH = 26, COMFUSE_OP_SIGMOID = 27,                                    /* unary: in0       */
  COMFUSE_OP_ADD = 32, COMFUSE_OP_SUB = 33, COMFUSE_OP_MUL = 34, COMFUSE_OP_DIV = 35,
  COMFUSE_OP_MAX = 36, COMFUSE_OP_MIN = 37,                                              /* binary: in0, in1 */
  /* reductions of in0 over the row (ReduceOp sum / prod / max / min and ReduceMode mean of the StreamReduction
   * node, Sec. 5); ARGMAX = lowest column attaining the row maximum, as a number */
  COMFUSE_OP_RED_SUM = 48, COMFUSE_OP_RED_MEAN = 49, COMFUSE_OP_RED_MAX = 50, COMFUSE_OP_RED_MIN = 51,
  COMFUSE_OP_RED_PROD = 52, COMFUSE_OP_RED_ARGMAX = 53,
  /* Top-K reduction (the StreamReduction node's hyper-parameter K, Sec. 5): `param` = K (1 .. 64, <= N).  The K largest
   * values of in0 per row in falling order, equal values in rising column order (VALUES), and their columns (INDICES).
   * K values per row: such a node can only be a row output (fp32 resp. int32 [batch*M, K]), not an input. */
  COMFUSE_OP_RED_TOPK_VALUES = 54, COMFUSE_OP_RED_TOPK_INDICES = 55
} comfuse_op_t;

typedef struct {
  int32_t op;        /* comfuse_op_t */
  int32_t in0, in1;  /* indices of earlier nodes, -1 where the op takes no such input */
  int32_t param;     /* ROWVEC / TENSOR: index into the parameter table; RED_TOPK_*: K; else -1 */
  float imm;         /* CONST: the value */
} comfuse_spec_node_t;

#define COMFUSE_SPEC_MAX_NODES 128
#define COMFUSE_SPEC_MAX_PARAMS 12
#define COMFUSE_SPEC_MAX_ROW_OUTPUTS 8

typedef struct {
  int32_t n_nodes;                   /* 1 .. COMFUSE_SPEC_MAX_NODES */
  const comfuse_spec_node_t* nodes;  /* HOST array, read during the call only */
  int32_t terminal;                  /* node whose value is Y */
  int32_t n_params;                  /* entries of the parameter table, 0 .. COMFUSE_SPEC_MAX_PARAMS */
  int32_t n_row_outputs;             /* 0 .. COMFUSE_SPEC_MAX_ROW_OUTPUTS */
  const int32_t* row_outputs;        /* HOST array of per-row valued nodes; output k is written to row_out[k]:
                                        fp32 [batch*M], or int32 [batch*M] when the node is a RED_ARGMAX;
                                        [batch*M, K] for the RED_TOPK_* nodes */
} comfuse_fusion_spec_t;

typedef struct {
  int32_t batch, M, N, K;
  int64_t lda, ldb, ldy;
  int64_t batch_stride_a, batch_stride_b, batch_stride_y;  /* used when batch > 1 */
  uint32_t flags;  /* 0, or COMFUSE_FLAG_B_ROW_MAJOR_NK: B stored [batch, N, K] (ldb >= K); any other bit: INVALID_ARG */
} comfuse_gemm_shape_t;

typedef enum {
  COMFUSE_SPEC_PATH_FUSED_KERNEL = 0,  /* a compiled fused instantiation (the enum kinds)                              */
  COMFUSE_SPEC_PATH_ROW_PROGRAM = 1,   /* GEMM kernel, bf16 Z, row-program kernel                                      */
  COMFUSE_SPEC_PATH_FUSED_PROGRAM = 2  /* ONE fused kernel whose epilogue interprets the program on-chip, stage by stage */
} comfuse_spec_path_t;

/* What the library will do with a program on a given shape (host-side analysis only; no device is touched). */
typedef struct {
  int32_t n_stages;       /* 1 + number of reductions on the longest dependency chain                    */
  int32_t n_reductions;   /* live reduction nodes                                                       */
  int32_t n_live_nodes;   /* nodes the terminal or a row output depends on                              */
  int32_t path;           /* comfuse_spec_path_t chosen when `fused` = 1                                */
  int32_t program_path;   /* the path when `fused` = 2 (compiled kinds skipped): FUSED_PROGRAM or ROW_PROGRAM */
  int32_t n_passes;       /* FUSED_PROGRAM: passes over the resident tensor                             */
  int32_t fused_kind;     /* FUSED_KERNEL: the comfuse_epilogue_kind_t it lowers to, else -1            */
  uint32_t fused_flags;   /* FUSED_KERNEL: COMFUSE_FLAG_* bits                                          */
  float alpha, eps, softcap;  /* FUSED_KERNEL: recovered constants                                      */
  int32_t causal;         /* FUSED_KERNEL: 1 if the program adds the causal mask                        */
  int32_t n_instructions; /* the row program (`fused` = 0): computed nodes the row kernel executes      */
  int32_t n_slots;        /* the row program: row-sized fp32 buffers held in shared memory at once      */
} comfuse_spec_plan_t;

/* Analyse a program: OK and *plan filled, INVALID_ARG for a malformed program (see above), UNSUPPORTED if it is valid
 * but cannot run on this shape (the row program's buffers exceed shared memory and no fused kernel matches). */
comfuse_status_t comfuse_spec_plan(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape,
                                   comfuse_spec_plan_t* plan);

/* Workspace comfuse_gemm_spec needs (bytes): 0 or row scratch for the fused kernel, batch*M*N*2 for the row program,
 * 0 for `fused` = 3. */
comfuse_status_t comfuse_gemm_spec_workspace_size(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape,
                                                  int32_t fused, size_t* bytes);

/* Whether programs can be compiled at run time on this machine: COMFUSE_OK, or COMFUSE_ERR_UNSUPPORTED with *why (may be
 * NULL) pointing at a static string that names what is missing (the toolkit's libnvrtc or its headers; CUDA_HOME is
 * searched, then /usr/local/cuda).  Touches no device. */
comfuse_status_t comfuse_program_compiler_status(const char** why);

/* Does whatever comfuse_gemm_spec(..., fused, ...) would do ahead of its first launch for this program and shape -- for
 * `fused` = 3, and for `fused` = 1 where that takes the generated form, it generates and compiles the kernel (no device
 * is needed for that; the module is loaded by the first launch) -- and nothing for the other pathways.  OK, the errors of comfuse_spec_plan, or UNSUPPORTED when `fused` = 3
 * and the program has no on-chip lowering, the shape no instantiation, or the compiler is not available. */
comfuse_status_t comfuse_gemm_spec_prepare(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, int32_t fused);

/* Y = program(A . B).  `params`: HOST array of spec->n_params DEVICE pointers (bf16; ROWVEC [N], TENSOR [batch, M, N]
 * with leading dimension param_ld[k], 0 = N); `param_ld` may be NULL.  `row_out`: HOST array of n_row_outputs DEVICE
 * pointers.  `fused` = 1: the best path (compiled fused kind, else the on-chip program -- as generated code where the run-time
 * compiler is available, else interpreted --, else row program); 2: skip the compiled kinds and interpret (on-chip
 * interpreter, else row program); 0: always the row-program pathway; 3: the kernel generated for
 * this program (UNSUPPORTED where the program has no on-chip lowering or the compiler is not available; no fallback).
 * Asynchronous on `cuda_stream`; the host arrays are not read after the call returns. */
comfuse_status_t comfuse_gemm_spec(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, const void* A,
                                   const void* B, void* Y, const void* const* params, const int64_t* param_ld,
                                   void* const* row_out, int32_t fused, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* COMFUSE_H_ */
