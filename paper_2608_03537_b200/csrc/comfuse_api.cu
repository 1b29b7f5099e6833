// C ABI of the library: argument validation, tensor-map construction, dispatch to the fused kernels or to the
// in-library unfused path.  Nothing here allocates device memory.
#include "../../include/comfuse.h"

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "b2b_params.h"
#include "host_common.h"
#include "row_params.h"

namespace comfuse {

__device__ unsigned int g_status_word = 0;

namespace {

std::atomic<uint64_t> g_launches{0};
std::mutex g_mutex;
constexpr int kMaxDev = 64;
DeviceInfo g_dev[kMaxDev];
std::atomic<bool> g_dev_ready[kMaxDev];  // zero-initialised: false

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;

EncodeFn get_encode_fn() {
  if (g_encode) return g_encode;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_encode) return g_encode;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  g_encode = reinterpret_cast<EncodeFn>(fn);
  return g_encode;
}

unsigned long long timeout_ns() {
  static unsigned long long v = [] {
    const char* e = std::getenv("COMFUSE_TIMEOUT_MS");
    long ms = e ? std::atol(e) : 2000;
    if (ms < 1) ms = 1;
    return static_cast<unsigned long long>(ms) * 1000000ull;
  }();
  return v;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool mult8(long long v) { return (v & 7) == 0; }

}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// COMFUSE_REDUCE_MODE=leader selects leader-follower aggregation of the row statistics, anything else all-to-all.
bool leader_reduce_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("COMFUSE_REDUCE_MODE");
    return e && std::strcmp(e, "leader") == 0;
  }();
  return on;
}

bool programmatic_launch_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("COMFUSE_PDL");
    return !(e && e[0] == '0');
  }();
  return on;
}

int split_row_block(int epi, int N, int K, long long row_pairs) {
  // COMFUSE_SPLIT_BLOCK=<width> forces the two-kernel form with that block width where N is a multiple of it (0 = never)
  static const int forced = [] {
    const char* e = std::getenv("COMFUSE_SPLIT_BLOCK");
    return e ? std::atoi(e) : -1;
  }();
  if (forced >= 0) return (forced > 0 && N > forced && N % forced == 0) ? forced : 0;
  // Measured (8192 rows; on-chip / two kernels with 256-column blocks, us): N = 4096: K = 4096 242 / 212, K = 1024 101 / 87,
  // K = 256 64 / 62 (LayerNorm 57 / 66); N = 2048: K = 4096 147 / 118, K = 1024 59 / 55; N = 1024, K = 4096: 55 / 69.
  // The clusters of 16 and 8 CTAs that hold rows of 4096 and 2048 columns fill 112 and 120 of the 148 SMs and cannot overlap
  // a tile's epilogue with the next MainLoop; the 256-column tiles of the two-kernel form can, on every SM.
  if (N >= 2048 && N % 256 == 0 && K >= 1024) return 256;
  const int form = norm_on_chip_form(N);
  if (form >= 2048 && form != N && K >= 1024) return 256;  // the same behind a row a little shorter than 2048 / 4096
  // Few rows behind a long contraction: the on-chip forms put one cluster on every pair of row blocks, which leaves most of
  // the machine idle when there are few pairs; 256-column tiles give N / 256 times as many work items.  Measured at 2048
  // rows (on chip / two kernels, us): N = 1024: K = 1024 20.3 / 16.7, K = 4096 48.0 / 32.2; at 8192 rows the clusters fill
  // the machine and the on-chip form is ahead again (K = 4096: 55 / 69).
  // (N = 512, 512 .. 4096 rows: K = 1536 LayerNorm 24 / 20, K = 2048 28 / 21, K = 4096 46 / 30; the RMSNorm kind gains from
  // K = 1024 on: 21 / 15; LayerNorm at K = 1024 is level.)
  if (std::getenv("COMFUSE_NO_SMALL_SPLIT") == nullptr && K >= (epi == EPI_LN ? 1536 : 1024) && N % 256 == 0 && N >= 512 && N <= 1024) {
    const long long cluster = N >= 768 ? 4 : 2;
    const long long two_kernel = row_pairs * (N / 256) * 2 < 148 ? row_pairs * (N / 256) * 2 : 148;
    if (row_pairs * cluster * 10 < two_kernel * 6) return 256;
  }
  // A row length that no single-kernel instantiation covers (1280, 1536, 2560, 3072, 5120, ...): the two-kernel form takes
  // any multiple of 256, at any K -- one fp16 trip of the row, which is still cheaper than the unfused path's bf16 Z plus
  // a row kernel.
  // 1280, 1536 and 1792 columns have on-chip forms too, on clusters of 10, 6 and 14 CTAs.  Measured (8192 rows; on chip / two
  // kernels, us; K = 256, 1024, 2048, 4096): LayerNorm N = 1280: 20 / 27, 29 / 38, 44 / 54, 75 / 87; N = 1536: 24 / 29, 39 / 40,
  // 58 / 57, 98 / 90; N = 1792: 30 / 33, 42 / 48, 67 / 70, 117 / 114.  RMSNorm N = 1280: 23 / 26, 30 / 37, 46 / 53, 77 / 86;
  // N = 1536: 27 / 28, 42 / 39, 61 / 55, 102 / 89; N = 1792: 36 / 32, 45 / 46, 70 / 69, 120 / 112.
  const bool ln = epi == EPI_LN;
  const bool more_rows = N == 1280 || (N == 1536 && K <= (ln ? 1024 : 256)) || (N == 1792 && ln && K <= 2048);
  const bool on_chip = form != 0 || more_rows;
  // (multiples of 4096: 4096-column blocks.)  N need not be a multiple of 256: the last tile is a partial one -- operands
  // outside the matrix read as zeros, stores are clipped, and the second kernel corrects that tile's statistic for them.
  return (!on_chip && N % kWideRowBlock != 0 && N <= 16 * kWideRowBlock) ? 256 : 0;
}

const DeviceInfo* current_device_info() {
  int d = -1;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDev) return nullptr;
  // g_dev_ready[d] is set (release) after every field of g_dev[d] has been written, so a thread that sees it (acquire)
  // sees the fields too.  The cached device addresses do not survive cudaDeviceReset.
  if (g_dev_ready[d].load(std::memory_order_acquire)) return &g_dev[d];
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_dev_ready[d].load(std::memory_order_relaxed)) return &g_dev[d];
  DeviceInfo info;
  if (cudaDeviceGetAttribute(&info.cc_major, cudaDevAttrComputeCapabilityMajor, d) != cudaSuccess) return nullptr;
  if (cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, d) != cudaSuccess) return nullptr;
  if (info.cc_major == 10) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_status_word) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    info.status_word = static_cast<unsigned int*>(addr);
  }
  info.device = d;
  g_dev[d] = info;
  g_dev_ready[d].store(true, std::memory_order_release);
  return &g_dev[d];
}

bool encode_tmap_bf16_3d(CUtensorMap* out, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                         uint64_t stride2_bytes, uint32_t box_rows) {
  EncodeFn enc = get_encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

// Tensor maps of a GEMM -> subgraph call.  R may be null (no residual): its map is then left zeroed and never used.
bool make_gemm_maps(GemmMaps* maps, const void* A, const void* B, const void* R, const void* Y, int batch, int M, int N, int K,
                    long long lda, long long ldb, long long ldr, long long ldy, long long bsa, long long bsb, long long bsr,
                    long long bsy, bool b_nk = false) {
  std::memset(maps, 0, sizeof(*maps));
  auto bs = [&](long long given, long long rows, long long ld) {
    return static_cast<uint64_t>(batch > 1 ? given : rows * ld) * 2;
  };
  if (!encode_tmap_bf16_3d(&maps->A, A, K, M, batch, static_cast<uint64_t>(lda) * 2, bs(bsa, M, lda), 128)) return false;
  if (b_nk) {  // B stored [N, K]: boxes of 64 rows (columns of the product) x 64 contraction elements
    if (!encode_tmap_bf16_3d(&maps->B, B, K, N, batch, static_cast<uint64_t>(ldb) * 2, bs(bsb, N, ldb), 64)) return false;
  } else if (!encode_tmap_bf16_3d(&maps->B, B, N, K, batch, static_cast<uint64_t>(ldb) * 2, bs(bsb, K, ldb), 64)) {
    return false;
  }
  if (!encode_tmap_bf16_3d(&maps->Y, Y, N, M, batch, static_cast<uint64_t>(ldy) * 2, bs(bsy, M, ldy), 32)) return false;
  if (R && !encode_tmap_bf16_3d(&maps->R, R, N, M, batch, static_cast<uint64_t>(ldr) * 2, bs(bsr, M, ldr), 128)) return false;
  return true;
}

comfuse_status_t check_device(const DeviceInfo** out) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return COMFUSE_ERR_CUDA;
  if (dev->cc_major != 10) return COMFUSE_ERR_ARCH;
  *out = dev;
  return COMFUSE_OK;
}

int kind_to_epi(int kind) {
  switch (kind) {
    case COMFUSE_EPI_BIAS_RES_LAYERNORM: return EPI_LN;
    case COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX: return EPI_RMS_MAX;
    case COMFUSE_EPI_SCALE_MASK_SOFTMAX: return EPI_SOFTMAX;
    default: return -1;
  }
}

comfuse_status_t validate_gemm_desc(const comfuse_gemm_desc_t* d) {
  if (!d) return COMFUSE_ERR_INVALID_ARG;
  if (d->batch < 1 || d->M < 1 || d->N < 1 || d->K < 1) return COMFUSE_ERR_INVALID_ARG;
  if (kind_to_epi(d->kind) < 0) return COMFUSE_ERR_INVALID_ARG;
  if (d->mask < COMFUSE_MASK_NONE || d->mask > COMFUSE_MASK_ADDITIVE) return COMFUSE_ERR_INVALID_ARG;
  if (d->fused != 0 && d->fused != 1) return COMFUSE_ERR_INVALID_ARG;
  if (d->reserved != 0) return COMFUSE_ERR_INVALID_ARG;
  if (d->flags & ~(COMFUSE_FLAG_POST_RELU | COMFUSE_FLAG_NO_ACTIVATION | COMFUSE_FLAG_B_ROW_MAJOR_NK)) return COMFUSE_ERR_INVALID_ARG;
  const bool b_nk = (d->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0;
  if ((d->flags & COMFUSE_FLAG_POST_RELU) && d->kind != COMFUSE_EPI_BIAS_RES_LAYERNORM) return COMFUSE_ERR_INVALID_ARG;
  if ((d->flags & COMFUSE_FLAG_NO_ACTIVATION) && d->kind != COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX) return COMFUSE_ERR_INVALID_ARG;
  if (!(d->softcap >= 0.f) || (d->softcap > 0.f && d->kind != COMFUSE_EPI_SCALE_MASK_SOFTMAX)) return COMFUSE_ERR_INVALID_ARG;
  if (d->lda < d->K || d->ldb < (b_nk ? d->K : d->N) || d->ldy < d->N) return COMFUSE_ERR_INVALID_ARG;
  if (d->kind != COMFUSE_EPI_SCALE_MASK_SOFTMAX && d->mask != COMFUSE_MASK_NONE) return COMFUSE_ERR_INVALID_ARG;
  if (!mult8(d->N) || !mult8(d->K)) return COMFUSE_ERR_ALIGNMENT;
  if (!mult8(d->lda) || !mult8(d->ldb) || !mult8(d->ldy)) return COMFUSE_ERR_ALIGNMENT;
  if (d->batch > 1) {
    if (d->batch_stride_a < static_cast<long long>(d->M - 1) * d->lda + d->K) return COMFUSE_ERR_INVALID_ARG;
    if (d->batch_stride_b < (b_nk ? static_cast<long long>(d->N - 1) * d->ldb + d->K : static_cast<long long>(d->K - 1) * d->ldb + d->N))
      return COMFUSE_ERR_INVALID_ARG;
    if (d->batch_stride_y < static_cast<long long>(d->M - 1) * d->ldy + d->N) return COMFUSE_ERR_INVALID_ARG;
    if (!mult8(d->batch_stride_a) || !mult8(d->batch_stride_b) || !mult8(d->batch_stride_y)) return COMFUSE_ERR_ALIGNMENT;
  }
  if (d->mask == COMFUSE_MASK_CAUSAL && d->M != d->N) return COMFUSE_ERR_UNSUPPORTED;
  return COMFUSE_OK;
}

// Does a fused instantiation exist for this description?  `on_chip_only`: without the two-kernel form.
comfuse_status_t fused_supported(const comfuse_gemm_desc_t* d, bool on_chip_only = false) {
  FusedParams p = {};
  p.b_nk = (d->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) ? 1 : 0;
  p.M = d->M;
  p.N = d->N;
  p.K = d->K;
  p.wide_block = on_chip_only ? 0 : wide_row_block(kind_to_epi(d->kind), d->N, d->K, static_cast<long long>(d->batch) * ((d->M + 255) / 256));
  p.wide = p.wide_block > 0;
  GemmMaps dummy;
  std::memset(&dummy, 0, sizeof(dummy));
  cudaError_t e = cudaErrorInvalidValue;
  switch (kind_to_epi(d->kind)) {
    case EPI_LN: e = launch_fused_layernorm(dummy, p, nullptr, true); break;
    case EPI_RMS_MAX: e = launch_fused_rmsnorm_max(dummy, p, nullptr, true); break;
    case EPI_SOFTMAX: e = launch_fused_softmax(dummy, p, nullptr, true); break;
    default: break;
  }
  return e == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_UNSUPPORTED;
}

}  // namespace

comfuse_status_t gemm_to_bf16(int batch, int M, int N, int K, long long lda, long long ldb, long long batch_stride_a,
                              long long batch_stride_b, const void* A, const void* B, void* Z, cudaStream_t st, bool b_nk) {
  const DeviceInfo* dev = nullptr;
  comfuse_status_t s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  GemmMaps maps;
  if (!make_gemm_maps(&maps, A, B, nullptr, Z, batch, M, N, K, lda, ldb, 0, N, batch_stride_a, batch_stride_b, 0,
                      static_cast<long long>(M) * N, b_nk))
    return COMFUSE_ERR_CUDA;
  FusedParams p = {};
  p.b_nk = b_nk ? 1 : 0;
  p.M = M; p.N = N; p.K = K; p.batch = batch;
  p.mblocks = (M + 127) / 128;
  p.nblocks = 1;
  p.total_tiles = batch * p.mblocks;
  p.alpha = 1.f;
  p.status = dev->status_word;
  p.timeout_ns = timeout_ns();
  p.Y = static_cast<uint16_t*>(Z);
  p.ldy = N;
  p.batch_stride_y = static_cast<long long>(M) * N;
  return launch_plain_gemm(maps, p, st) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

comfuse_status_t run_gemm_elementwise(int batch, int M, int N, int K, long long lda, long long ldb, long long ldy, long long batch_stride_a,
                                      long long batch_stride_b, long long batch_stride_y, const void* A, const void* B, void* Y,
                                      const void* bias, float alpha, int activation, cudaStream_t st, bool b_nk) {
  const DeviceInfo* dev = nullptr;
  comfuse_status_t s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  GemmMaps maps;
  if (!make_gemm_maps(&maps, A, B, nullptr, Y, batch, M, N, K, lda, ldb, 0, ldy, batch_stride_a, batch_stride_b, 0,
                      batch > 1 ? batch_stride_y : 0, b_nk))
    return COMFUSE_ERR_CUDA;
  FusedParams p = {};
  p.b_nk = b_nk ? 1 : 0;
  p.M = M; p.N = N; p.K = K; p.batch = batch;
  p.mblocks = (M + 127) / 128;
  p.nblocks = 1;
  p.total_tiles = batch * p.mblocks;
  p.alpha = alpha;
  p.activation = activation;
  p.bias = static_cast<const uint16_t*>(bias);
  p.status = dev->status_word;
  p.timeout_ns = timeout_ns();
  p.Y = static_cast<uint16_t*>(Y);
  p.ldy = ldy;
  p.batch_stride_y = batch > 1 ? batch_stride_y : 0;
  return launch_gemm_elementwise(maps, p, st) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

comfuse_status_t run_fused_program(int batch, int M, int N, int K, long long lda, long long ldb, long long ldy, long long batch_stride_a,
                                   long long batch_stride_b, long long batch_stride_y, const void* A, const void* B, void* Y,
                                   const StageProgram& prog, const void* const vecs[3], const void* residual, long long ldr,
                                   cudaStream_t st, bool query_only, bool b_nk, bool compiled) {
  FusedParams p = {};
  p.M = M; p.N = N; p.K = K; p.batch = batch;
  p.b_nk = b_nk ? 1 : 0;
  p.program = prog;  // (the query looks at it too: a program with temporaries runs as generated code only)
  GemmMaps maps;
  if (query_only) {
    std::memset(&maps, 0, sizeof(maps));
    const cudaError_t e = compiled ? launch_compiled_program(maps, p, nullptr, true, false) : launch_fused_program(maps, p, nullptr, true);
    return e == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_UNSUPPORTED;
  }
  const DeviceInfo* dev = nullptr;
  comfuse_status_t s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  const long long bsr = static_cast<long long>(M) * ldr;
  if (!make_gemm_maps(&maps, A, B, residual, Y, batch, M, N, K, lda, ldb, ldr, ldy, batch_stride_a, batch_stride_b, bsr,
                      batch > 1 ? batch_stride_y : 0, b_nk))
    return COMFUSE_ERR_CUDA;
  p.mblocks = (M + 127) / 128;
  p.nblocks = 1;
  p.total_tiles = batch * p.mblocks;
  p.alpha = 1.f;
  p.status = dev->status_word;
  p.timeout_ns = timeout_ns();
  p.leader_reduce = leader_reduce_enabled() ? 1 : 0;
  p.bias = static_cast<const uint16_t*>(vecs[0]);
  p.gamma = static_cast<const uint16_t*>(vecs[1]);
  p.beta = static_cast<const uint16_t*>(vecs[2]);
  p.residual = static_cast<const uint16_t*>(residual);
  p.ldr = ldr; p.batch_stride_r = bsr;
  p.Y = static_cast<uint16_t*>(Y);
  p.ldy = ldy; p.batch_stride_y = batch > 1 ? batch_stride_y : 0;
  p.program = prog;
  if (compiled) {
    const cudaError_t e = launch_compiled_program(maps, p, st, false, true);
    return e == cudaSuccess ? COMFUSE_OK : (e == cudaErrorInvalidValue ? COMFUSE_ERR_UNSUPPORTED : COMFUSE_ERR_CUDA);
  }
  return launch_fused_program(maps, p, st, false) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

comfuse_status_t prepare_compiled_program(int N, const StageProgram& prog) {
  FusedParams p = {};
  p.N = N;
  p.program = prog;
  GemmMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  return launch_compiled_program(maps, p, nullptr, false, false) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_UNSUPPORTED;
}

}  // namespace comfuse

using namespace comfuse;

extern "C" {

const char* comfuse_status_string(comfuse_status_t s) {
  switch (s) {
    case COMFUSE_OK: return "ok";
    case COMFUSE_ERR_INVALID_ARG: return "invalid argument";
    case COMFUSE_ERR_UNSUPPORTED: return "unsupported shape or op list for the fused path";
    case COMFUSE_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
    case COMFUSE_ERR_WORKSPACE: return "workspace missing or too small";
    case COMFUSE_ERR_ARCH: return "device is not compute capability 10.x";
    case COMFUSE_ERR_CUDA: return "CUDA call failed";
    case COMFUSE_ERR_TIMEOUT: return "bounded device-side wait expired";
    case COMFUSE_ERR_BOUNDS: return "a bounds predicate of the checked build failed (access skipped)";
    default: return "unknown status";
  }
}

uint64_t comfuse_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

comfuse_status_t comfuse_workspace_size(const comfuse_gemm_desc_t* desc, size_t* bytes) {
  if (!bytes) return COMFUSE_ERR_INVALID_ARG;
  comfuse_status_t s = validate_gemm_desc(desc);
  if (s != COMFUSE_OK) return s;
  if (desc->fused) {
    s = fused_supported(desc);
    if (s != COMFUSE_OK) return s;
    // rows wider than one cluster: one partial statistic (8 bytes) per row and 4096-column block
    *bytes = static_cast<size_t>(wide_row_blocks(kind_to_epi(desc->kind), desc->N, desc->K, static_cast<long long>(desc->batch) * ((desc->M + 255) / 256))) *
             desc->batch * desc->M * sizeof(float2);
  } else {
    if (desc->N > 8192) return COMFUSE_ERR_UNSUPPORTED;
    *bytes = static_cast<size_t>(desc->batch) * desc->M * desc->N * 2;  // dense bf16 Z
  }
  return COMFUSE_OK;
}

comfuse_status_t comfuse_gemm_epilogue(const comfuse_gemm_desc_t* desc, const void* A, const void* B, void* Y,
                                       const comfuse_epilogue_args_t* args, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
  comfuse_status_t s = validate_gemm_desc(desc);
  if (s != COMFUSE_OK) return s;
  if (!A || !B || !Y) return COMFUSE_ERR_INVALID_ARG;
  comfuse_epilogue_args_t a;
  std::memset(&a, 0, sizeof(a));
  if (args) a = *args;
  const int epi = kind_to_epi(desc->kind);
  if (epi == EPI_RMS_MAX && (!a.row_max || !a.row_argmax)) return COMFUSE_ERR_INVALID_ARG;
  if (desc->mask == COMFUSE_MASK_ADDITIVE && !a.mask) return COMFUSE_ERR_INVALID_ARG;
  if (a.residual && (desc->ldr < desc->N || !mult8(desc->ldr) ||
                     (desc->batch > 1 && (!mult8(desc->batch_stride_r) ||
                                          desc->batch_stride_r < static_cast<long long>(desc->M - 1) * desc->ldr + desc->N))))
    return desc->ldr < desc->N ? COMFUSE_ERR_INVALID_ARG : COMFUSE_ERR_ALIGNMENT;
  if (!aligned16(A) || !aligned16(B) || !aligned16(Y) || !aligned16(a.bias) || !aligned16(a.residual) ||
      !aligned16(a.gamma) || !aligned16(a.beta) || !aligned16(a.mask))
    return COMFUSE_ERR_ALIGNMENT;

  size_t need = 0;
  s = comfuse_workspace_size(desc, &need);
  if (s != COMFUSE_OK) return s;
  // For rows that fit a cluster (N <= 4096) the two-kernel form is an optimisation, not a need: a fused call that brings no
  // (or too small a) workspace keeps the row on chip instead of being refused.
  const bool split_optional = desc->fused && desc->N <= kWideRowBlock && need > 0 && fused_supported(desc, true) == COMFUSE_OK;
  const bool have_ws = workspace && workspace_bytes >= need && aligned16(workspace);
  if (split_optional && !have_ws) need = 0;
  if (need > 0 && (!workspace || workspace_bytes < need)) return COMFUSE_ERR_WORKSPACE;
  if (need > 0 && !aligned16(workspace)) return COMFUSE_ERR_ALIGNMENT;

  const DeviceInfo* dev = nullptr;
  s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  const long long bsr = desc->batch > 1 ? desc->batch_stride_r : 0;
  const long long bsy = desc->batch > 1 ? desc->batch_stride_y : 0;
  const bool b_nk = (desc->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0;
  GemmMaps maps;
  if (desc->fused) {
    if (!make_gemm_maps(&maps, A, B, a.residual, Y, desc->batch, desc->M, desc->N, desc->K, desc->lda, desc->ldb, desc->ldr,
                        desc->ldy, desc->batch_stride_a, desc->batch_stride_b, bsr, bsy, b_nk))
      return COMFUSE_ERR_CUDA;
  } else {  // the GEMM's output is the dense bf16 Z in the workspace
    if (!make_gemm_maps(&maps, A, B, nullptr, workspace, desc->batch, desc->M, desc->N, desc->K, desc->lda, desc->ldb, 0, desc->N,
                        desc->batch_stride_a, desc->batch_stride_b, 0, static_cast<long long>(desc->M) * desc->N, b_nk))
      return COMFUSE_ERR_CUDA;
  }

  FusedParams p = {};
  p.M = desc->M; p.N = desc->N; p.K = desc->K; p.batch = desc->batch;
  p.mblocks = (desc->M + 127) / 128;
  p.nblocks = 1;
  p.total_tiles = p.batch * p.mblocks;
  p.alpha = desc->alpha; p.eps = desc->eps;
  p.causal = desc->mask == COMFUSE_MASK_CAUSAL;
  p.b_nk = b_nk ? 1 : 0;  // every GEMM kernel reads the operand as stored
  p.post_relu = (desc->flags & COMFUSE_FLAG_POST_RELU) ? 1 : 0;
  p.no_activation = (desc->flags & COMFUSE_FLAG_NO_ACTIVATION) ? 1 : 0;
  p.softcap = desc->softcap;
  p.status = dev->status_word;
  p.timeout_ns = timeout_ns();
  p.leader_reduce = leader_reduce_enabled() ? 1 : 0;
#ifdef COMFUSE_TRACE
  // tracing build: COMFUSE_TRACE_PTR holds the device address of a uint64[64] buffer for phase timestamps
  if (const char* tp = std::getenv("COMFUSE_TRACE_PTR")) p.trace = reinterpret_cast<unsigned long long*>(std::strtoull(tp, nullptr, 0));
  if (const char* tf = std::getenv("COMFUSE_TRACE_FLAGS")) p.trace_flags = std::atoi(tf);
#endif

  cudaError_t e;
  if (desc->fused) {
    p.bias = static_cast<const uint16_t*>(a.bias);
    p.gamma = static_cast<const uint16_t*>(a.gamma);
    p.beta = static_cast<const uint16_t*>(a.beta);
    p.residual = static_cast<const uint16_t*>(a.residual);
    p.ldr = desc->ldr; p.batch_stride_r = bsr;
    p.Y = static_cast<uint16_t*>(Y);
    p.ldy = desc->ldy; p.batch_stride_y = bsy;
    p.row_max = a.row_max; p.row_argmax = a.row_argmax;
    p.mask = desc->mask == COMFUSE_MASK_ADDITIVE ? static_cast<const uint16_t*>(a.mask) : nullptr;
    const long long row_pairs = static_cast<long long>(desc->batch) * ((desc->M + 255) / 256);
    const int wide_blocks = need > 0 ? wide_row_blocks(epi, desc->N, desc->K, row_pairs) : 0;
    if (wide_blocks) {
      p.wide_block = wide_row_block(epi, desc->N, desc->K, row_pairs);  // first kernel: per-block stage 1, un-normalised x to Y, partial statistics to the workspace
      p.wide = 1;
      p.nblocks = wide_blocks;
      p.wide_partials = static_cast<float2*>(workspace);
      p.gamma = nullptr;
      p.beta = nullptr;
    }
    switch (epi) {
      case EPI_LN: e = launch_fused_layernorm(maps, p, st, false); break;
      case EPI_RMS_MAX: e = launch_fused_rmsnorm_max(maps, p, st, false); break;
      default: e = launch_fused_softmax(maps, p, st, false); break;
    }
    if (e == cudaSuccess && wide_blocks) {  // second kernel: merge the blocks' statistics, rescale the row in place
      RowParams r = {};
      r.batch = desc->batch; r.M = desc->M; r.N = desc->N;
      r.gamma = static_cast<const uint16_t*>(a.gamma);
      r.beta = static_cast<const uint16_t*>(a.beta);
      r.eps = desc->eps;
      r.post_relu = p.post_relu;
      r.Y = static_cast<uint16_t*>(Y);
      r.ldy = desc->ldy; r.batch_stride_y = bsy;
      r.row_max = a.row_max; r.row_argmax = a.row_argmax;
      e = launch_wide_row_finish(epi, r, p.wide_partials, wide_blocks, p.wide_block, st);
    }
    return e == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
  }

  // unfused: GEMM writes dense bf16 Z [batch, M, N] into the workspace, a row kernel finishes
  p.Y = static_cast<uint16_t*>(workspace);
  p.ldy = desc->N;
  p.batch_stride_y = static_cast<long long>(desc->M) * desc->N;
  e = launch_plain_gemm(maps, p, st);
  if (e != cudaSuccess) return COMFUSE_ERR_CUDA;
  RowParams r = {};
  r.batch = desc->batch; r.M = desc->M; r.N = desc->N;
  r.Z = static_cast<const uint16_t*>(workspace);
  r.ldz = desc->N; r.batch_stride_z = static_cast<long long>(desc->M) * desc->N;
  r.bias = static_cast<const uint16_t*>(a.bias);
  r.gamma = static_cast<const uint16_t*>(a.gamma);
  r.beta = static_cast<const uint16_t*>(a.beta);
  r.residual = static_cast<const uint16_t*>(a.residual);
  r.ldr = desc->ldr; r.batch_stride_r = bsr;
  r.mask = desc->mask == COMFUSE_MASK_ADDITIVE ? static_cast<const uint16_t*>(a.mask) : nullptr;
  r.causal = p.causal;
  r.alpha = desc->alpha; r.eps = desc->eps;
  r.post_relu = p.post_relu; r.no_activation = p.no_activation; r.softcap = desc->softcap;
  r.Y = static_cast<uint16_t*>(Y);
  r.ldy = desc->ldy; r.batch_stride_y = bsy;
  r.row_max = a.row_max; r.row_argmax = a.row_argmax;
  e = launch_row_epilogue(epi, r, st);
  return e == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

static comfuse_status_t validate_b2b_desc(const comfuse_b2b_desc_t* d) {
  if (!d) return COMFUSE_ERR_INVALID_ARG;
  if (d->M < 1 || d->K < 1 || d->N1 < 1 || d->N2 < 1) return COMFUSE_ERR_INVALID_ARG;
  if (d->fused != 0 && d->fused != 1) return COMFUSE_ERR_INVALID_ARG;
  if (d->kind != COMFUSE_B2B_MLP_GELU_LAYERNORM && d->kind != COMFUSE_B2B_SOFTMAX_ATTENTION && d->kind != COMFUSE_B2B_MLP_RELU)
    return COMFUSE_ERR_INVALID_ARG;
  if (d->batch < 1 || (d->flags & ~COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR) != 0) return COMFUSE_ERR_INVALID_ARG;
  if (d->flags != 0 && d->kind != COMFUSE_B2B_SOFTMAX_ATTENTION) return COMFUSE_ERR_INVALID_ARG;
  if (d->kind == COMFUSE_B2B_MLP_GELU_LAYERNORM) {
    if (d->batch != 1) return COMFUSE_ERR_INVALID_ARG;
    if (d->N2 != d->K) return COMFUSE_ERR_INVALID_ARG;  // the residual is X itself
  } else if (d->kind == COMFUSE_B2B_MLP_RELU) {
    if (d->batch != 1) return COMFUSE_ERR_INVALID_ARG;
  } else if (!(d->alpha > 0.f)) {
    return COMFUSE_ERR_INVALID_ARG;
  }
  if (!mult8(d->K) || !mult8(d->N1) || !mult8(d->N2)) return COMFUSE_ERR_ALIGNMENT;
  if (d->kind == COMFUSE_B2B_MLP_RELU) {
    if (d->fused && !b2b_stream_supported(d->K, d->N1, d->N2)) return COMFUSE_ERR_UNSUPPORTED;
    return COMFUSE_OK;  // unfused: two calls of the reduction-free GEMM kind, any N1 / N2
  }
  if (d->fused && !b2b_fused_supported(d->K, d->N1, d->N2, d->kind)) return COMFUSE_ERR_UNSUPPORTED;
  if (!d->fused && (d->kind == COMFUSE_B2B_MLP_GELU_LAYERNORM ? d->N2 : d->N1) > 8192) return COMFUSE_ERR_UNSUPPORTED;
  return COMFUSE_OK;
}

comfuse_status_t comfuse_b2b_workspace_size(const comfuse_b2b_desc_t* desc, size_t* bytes) {
  if (!bytes) return COMFUSE_ERR_INVALID_ARG;
  comfuse_status_t s = validate_b2b_desc(desc);
  if (s != COMFUSE_OK) return s;
  if (desc->kind == COMFUSE_B2B_SOFTMAX_ATTENTION)  // unfused: the bf16 scores / probabilities [batch, M, N1]
    *bytes = desc->fused ? 0
                         : static_cast<size_t>(desc->batch) * desc->M * desc->N1 * 2;
  else if (desc->kind == COMFUSE_B2B_MLP_RELU)  // unfused: the bf16 hidden layer [M, N1]
    *bytes = desc->fused ? 0 : static_cast<size_t>(desc->M) * desc->N1 * 2;
  else
    *bytes = desc->fused ? 0 : (static_cast<size_t>(desc->M) * desc->N1 + static_cast<size_t>(desc->M) * desc->N2) * 2;
  return COMFUSE_OK;
}

comfuse_status_t comfuse_b2b_gemm(const comfuse_b2b_desc_t* desc, const void* X, const void* W1, const void* b1,
                                  const void* W2, const void* b2, const void* gamma, const void* beta, void* O,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  comfuse_status_t s = validate_b2b_desc(desc);
  if (s != COMFUSE_OK) return s;
  if (!X || !W1 || !W2 || !O) return COMFUSE_ERR_INVALID_ARG;
  const bool attention = desc->kind == COMFUSE_B2B_SOFTMAX_ATTENTION;
  if (attention && (b1 || b2 || gamma || beta)) return COMFUSE_ERR_INVALID_ARG;
  const bool relu_mlp = desc->kind == COMFUSE_B2B_MLP_RELU;
  if (relu_mlp && (gamma || beta)) return COMFUSE_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W1) || !aligned16(W2) || !aligned16(O) || !aligned16(b1) || !aligned16(b2) ||
      !aligned16(gamma) || !aligned16(beta))
    return COMFUSE_ERR_ALIGNMENT;
  size_t need = 0;
  s = comfuse_b2b_workspace_size(desc, &need);
  if (s != COMFUSE_OK) return s;
  if (need > 0 && (!workspace || workspace_bytes < need)) return COMFUSE_ERR_WORKSPACE;
  if (need > 0 && !aligned16(workspace)) return COMFUSE_ERR_ALIGNMENT;
  const DeviceInfo* dev = nullptr;
  s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int M = desc->M, K = desc->K, N1 = desc->N1, N2 = desc->N2;

  if (desc->fused) {
    B2bParams bp = {};
    bp.M = M; bp.K = K; bp.N1 = N1; bp.N2 = N2;
    bp.batch = desc->batch; bp.mode = attention ? 1 : (relu_mlp ? 2 : 0); bp.alpha = desc->alpha;
    bp.keys_row_major = (desc->flags & COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR) ? 1 : 0;
    bp.eps = desc->eps;
    bp.X = static_cast<const uint16_t*>(X);
    bp.b1 = static_cast<const uint16_t*>(b1);
    bp.b2 = static_cast<const uint16_t*>(b2);
    bp.gamma = static_cast<const uint16_t*>(gamma);
    bp.beta = static_cast<const uint16_t*>(beta);
    bp.O = static_cast<uint16_t*>(O);
    bp.status = dev->status_word;
    bp.timeout_ns = timeout_ns();
#ifdef COMFUSE_TRACE
    if (const char* tp = std::getenv("COMFUSE_TRACE_PTR")) bp.trace = reinterpret_cast<unsigned long long*>(std::strtoull(tp, nullptr, 0));
    if (const char* tf = std::getenv("COMFUSE_TRACE_FLAGS")) bp.trace_flags = std::atoi(tf);
#endif
    cudaError_t e = relu_mlp ? launch_b2b_stream(X, W1, W2, bp, st)
                    : attention ? launch_b2b_fused(X, W1, W2, bp, st)
                                : launch_b2b_mlp(X, W1, W2, bp, st);
    return e == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
  }

  if (relu_mlp) {
    // unfused: S = ReLU(X.W1 + b1) as bf16 in the workspace, then O = ReLU(S.W2 + b2): the reduction-free GEMM kind twice
    s = run_gemm_elementwise(1, M, N1, K, K, N1, N1, 0, 0, 0, X, W1, workspace, b1, 1.f, COMFUSE_OP_RELU, st);
    if (s != COMFUSE_OK) return s;
    return run_gemm_elementwise(1, M, N2, N1, N1, N2, N2, 0, 0, 0, workspace, W2, O, b2, 1.f, COMFUSE_OP_RELU, st);
  }

  if (attention) {
    // unfused: P = X.W1 (bf16, workspace) -> row softmax of alpha * P in place -> O = P.W2, batched
    uint16_t* P = static_cast<uint16_t*>(workspace);
    const int nb = desc->batch;
    const bool keys_rm = (desc->flags & COMFUSE_B2B_FLAG_KEYS_ROW_MAJOR) != 0;  // keys [nb, N1, K]: the plain GEMM reads them as stored
    GemmMaps maps;
    FusedParams p = {};
    p.batch = nb; p.mblocks = (M + 127) / 128; p.alpha = 1.f;
    p.status = dev->status_word; p.timeout_ns = timeout_ns();
    if (!make_gemm_maps(&maps, X, W1, nullptr, P, nb, M, N1, K, K, keys_rm ? K : N1, 0, N1, static_cast<long long>(M) * K,
                        static_cast<long long>(K) * N1, 0, static_cast<long long>(M) * N1, keys_rm))
      return COMFUSE_ERR_CUDA;
    p.b_nk = keys_rm ? 1 : 0;
    p.M = M; p.N = N1; p.K = K; p.Y = P; p.ldy = N1; p.batch_stride_y = static_cast<long long>(M) * N1;
    if (launch_plain_gemm(maps, p, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    RowParams r = {};
    r.batch = 1; r.M = nb * M; r.N = N1;  // the rows of all batches, dense
    r.Z = P; r.ldz = N1;
    r.alpha = desc->alpha;
    r.Y = P; r.ldy = N1;
    if (launch_row_epilogue(EPI_SOFTMAX, r, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    if (!make_gemm_maps(&maps, P, W2, nullptr, O, nb, M, N2, N1, N1, N2, 0, N2, static_cast<long long>(M) * N1,
                        static_cast<long long>(N1) * N2, 0, static_cast<long long>(M) * N2))
      return COMFUSE_ERR_CUDA;
    p.b_nk = 0;
    p.N = N2; p.K = N1; p.Y = static_cast<uint16_t*>(O); p.ldy = N2; p.batch_stride_y = static_cast<long long>(M) * N2;
    return launch_plain_gemm(maps, p, st) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
  }

  // unfused: P = X.W1 -> S = GELU(P + b1) in place -> O' = S.W2 -> LayerNorm(O' + b2 + X)
  uint16_t* P = static_cast<uint16_t*>(workspace);
  uint16_t* Op = P + static_cast<size_t>(M) * N1;
  GemmMaps maps;
  FusedParams p = {};
  p.batch = 1; p.mblocks = (M + 127) / 128; p.alpha = 1.f;
  p.status = dev->status_word; p.timeout_ns = timeout_ns();
  if (!make_gemm_maps(&maps, X, W1, nullptr, P, 1, M, N1, K, K, N1, 0, N1, 0, 0, 0, 0)) return COMFUSE_ERR_CUDA;
  p.M = M; p.N = N1; p.K = K; p.Y = P; p.ldy = N1;
  if (launch_plain_gemm(maps, p, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (launch_bias_gelu(P, static_cast<const uint16_t*>(b1), M, N1, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (!make_gemm_maps(&maps, P, W2, nullptr, Op, 1, M, N2, N1, N1, N2, 0, N2, 0, 0, 0, 0)) return COMFUSE_ERR_CUDA;
  p.N = N2; p.K = N1; p.Y = Op; p.ldy = N2;
  if (launch_plain_gemm(maps, p, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  RowParams r = {};
  r.batch = 1; r.M = M; r.N = N2;
  r.Z = Op; r.ldz = N2;
  r.bias = static_cast<const uint16_t*>(b2);
  r.gamma = static_cast<const uint16_t*>(gamma);
  r.beta = static_cast<const uint16_t*>(beta);
  r.residual = static_cast<const uint16_t*>(X); r.ldr = K;
  r.alpha = 1.f; r.eps = desc->eps;
  r.Y = static_cast<uint16_t*>(O); r.ldy = N2;
  return launch_row_epilogue(EPI_LN, r, st) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

comfuse_status_t comfuse_last_device_status(void* cuda_stream) {
  const DeviceInfo* dev = nullptr;
  comfuse_status_t s = check_device(&dev);
  if (s != COMFUSE_OK) return s;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return COMFUSE_ERR_CUDA;
  unsigned int word = 0;
  if (cudaMemcpy(&word, dev->status_word, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (word != 0) {
    const unsigned int zero = 0;
    if (cudaMemcpy(dev->status_word, &zero, sizeof(zero), cudaMemcpyHostToDevice) != cudaSuccess) return COMFUSE_ERR_CUDA;
    return (word & 1u) ? COMFUSE_ERR_TIMEOUT : COMFUSE_ERR_BOUNDS;
  }
  return COMFUSE_OK;
}

}  // extern "C"
