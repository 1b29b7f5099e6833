// Host-buffer forms of the two entry points: the per-step tensors (activations in, result out) are HOST pointers; the
// call copies them to / from a device staging area the caller provides and runs the same kernels in between, all on the
// caller's stream.  Nothing is allocated; the staging layout keeps the tensors' own strides, so every copy is one
// contiguous cudaMemcpyAsync of the tensor's extent.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <mutex>

#include "../../include/comfuse.h"

namespace {

// Row-chunk pipelining of the host-buffer GEMM call: rows are independent, so the call is cut into up to kPipeChunks row
// ranges; range c's inputs are copied on a copy-in stream while range c-1 computes on the caller's stream and range c-2's
// result goes back on a copy-out stream (both copy engines and the SMs busy at once).  The two helper streams and the
// events are created once per device and reused; the caller's stream forks into them at the start of the call and joins
// them at its end, so the call keeps its stream-ordered semantics.  COMFUSE_HOST_PIPELINE=0 turns it off.
constexpr int kPipeChunks = 32;   // events held per device; the default cut is kPipeDefault ranges (COMFUSE_HOST_CHUNKS=<n> overrides it)
constexpr int kPipeDefault = 8;
// Every range costs host time (tensor-map encodes, launches, event records): cut only into ranges whose host -> device
// traffic is worth it.
constexpr size_t kPipeMinChunkBytes = 4u << 20;
int pipe_chunks(size_t h2d_bytes) {
  static const int most = [] {
    const char* e = std::getenv("COMFUSE_HOST_CHUNKS");
    const int v = e ? std::atoi(e) : 0;
    return v >= 2 && v <= kPipeChunks ? v : kPipeDefault;
  }();
  const size_t n = h2d_bytes / kPipeMinChunkBytes;
  return n >= static_cast<size_t>(most) ? most : static_cast<int>(n);
}
constexpr int kMaxDevPipe = 64;
struct Pipe {
  bool ready = false;
  std::mutex use;  // held by a call while it enqueues: the helper streams and events serve one call at a time
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, copied[kPipeChunks] = {}, computed[kPipeChunks] = {};
};
Pipe g_pipe[kMaxDevPipe];
std::mutex g_pipe_mutex;

Pipe* pipe_for_current_device() {
  static const bool enabled = [] {
    const char* e = std::getenv("COMFUSE_HOST_PIPELINE");
    return !(e && e[0] == '0');
  }();
  int d = -1;
  if (!enabled || cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevPipe) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  Pipe& p = g_pipe[d];
  if (p.ready) return &p;
  bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.join, cudaEventDisableTiming) == cudaSuccess;
  for (int c = 0; ok && c < kPipeChunks; ++c)
    ok = cudaEventCreateWithFlags(&p.copied[c], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&p.computed[c], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) return nullptr;
  p.ready = true;
  return &p;
}

constexpr size_t kAlign = 256;
size_t round_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

// bytes spanned by a [batch, rows, cols] bf16 tensor with leading dimension ld and batch stride bs (elements)
size_t extent_bytes(int batch, int rows, int cols, long long ld, long long bs) {
  const long long last = static_cast<long long>(rows - 1) * ld + cols;
  return static_cast<size_t>((batch > 1 ? static_cast<long long>(batch - 1) * bs : 0) + last) * 2;
}

struct Extents { size_t a, b, r, y; };

Extents extents_of(const comfuse_gemm_desc_t* d, uint32_t mask) {
  Extents e = {0, 0, 0, 0};
  if (mask & COMFUSE_HOST_A) e.a = extent_bytes(d->batch, d->M, d->K, d->lda, d->batch_stride_a);
  if (mask & COMFUSE_HOST_B)  // stored [K, N], or [N, K] with COMFUSE_FLAG_B_ROW_MAJOR_NK
    e.b = (d->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) ? extent_bytes(d->batch, d->N, d->K, d->ldb, d->batch_stride_b)
                                                   : extent_bytes(d->batch, d->K, d->N, d->ldb, d->batch_stride_b);
  if (mask & COMFUSE_HOST_RESIDUAL) e.r = extent_bytes(d->batch, d->M, d->N, d->ldr, d->batch_stride_r);
  if (mask & COMFUSE_HOST_Y) e.y = extent_bytes(d->batch, d->M, d->N, d->ldy, d->batch_stride_y);
  return e;
}

}  // namespace

extern "C" comfuse_status_t comfuse_host_staging_size(const comfuse_gemm_desc_t* desc, uint32_t host_mask, size_t* bytes) {
  if (!desc || !bytes) return COMFUSE_ERR_INVALID_ARG;
  if (host_mask & ~(COMFUSE_HOST_A | COMFUSE_HOST_B | COMFUSE_HOST_RESIDUAL | COMFUSE_HOST_Y)) return COMFUSE_ERR_INVALID_ARG;
  size_t ws = 0;
  const comfuse_status_t s = comfuse_workspace_size(desc, &ws);  // validates the description
  if (s != COMFUSE_OK) return s;
  if ((host_mask & COMFUSE_HOST_RESIDUAL) && desc->ldr < desc->N) return COMFUSE_ERR_INVALID_ARG;
  const Extents e = extents_of(desc, host_mask);
  *bytes = round_up(e.a) + round_up(e.b) + round_up(e.r) + round_up(e.y);
  return COMFUSE_OK;
}

extern "C" comfuse_status_t comfuse_gemm_epilogue_host(const comfuse_gemm_desc_t* desc, const void* A, const void* B, void* Y,
                                                       const comfuse_epilogue_args_t* args, uint32_t host_mask,
                                                       void* staging, size_t staging_bytes, void* workspace,
                                                       size_t workspace_bytes, void* cuda_stream) {
  size_t need = 0;
  comfuse_status_t s = comfuse_host_staging_size(desc, host_mask, &need);
  if (s != COMFUSE_OK) return s;
  if (!A || !B || !Y) return COMFUSE_ERR_INVALID_ARG;
  if ((host_mask & COMFUSE_HOST_RESIDUAL) && !(args && args->residual)) return COMFUSE_ERR_INVALID_ARG;
  if (need > 0 && (!staging || staging_bytes < need)) return COMFUSE_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(staging) & 15u) return COMFUSE_ERR_ALIGNMENT;
  {  // everything that can be checked on the host is checked before the first copy is enqueued
    size_t ws_all = 0;
    if (comfuse_workspace_size(desc, &ws_all) != COMFUSE_OK) return COMFUSE_ERR_INVALID_ARG;
    if (ws_all > 0 && (!workspace || workspace_bytes < ws_all)) return COMFUSE_ERR_WORKSPACE;
    if (ws_all > 0 && (reinterpret_cast<uintptr_t>(workspace) & 15u)) return COMFUSE_ERR_ALIGNMENT;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Extents e = extents_of(desc, host_mask);
  unsigned char* cur = static_cast<unsigned char*>(staging);
  const void* dA = A;
  const void* dB = B;
  void* dY = Y;
  comfuse_epilogue_args_t a = {};
  if (args) a = *args;
  auto stage_in = [&](const void* host, size_t bytes, const void** dev_ptr) {
    *dev_ptr = cur;
    const cudaError_t err = cudaMemcpyAsync(cur, host, bytes, cudaMemcpyHostToDevice, st);
    cur += round_up(bytes);
    return err == cudaSuccess;
  };
  // ---- pipelined form: one row range after the other (row-independent op lists, one batch, A and Y in host memory)
  const int nchunks = pipe_chunks(e.a + e.r);
  const int rows_per_chunk = nchunks >= 2 ? ((desc->M + nchunks - 1) / nchunks + 255) / 256 * 256 : desc->M;
  Pipe* pipe = (nchunks >= 2 && desc->batch == 1 && desc->kind != COMFUSE_EPI_SCALE_MASK_SOFTMAX && (host_mask & COMFUSE_HOST_A) &&
                (host_mask & COMFUSE_HOST_Y) && desc->M >= 2 * rows_per_chunk)
                   ? pipe_for_current_device() : nullptr;
  if (pipe) {
    std::lock_guard<std::mutex> one_call(pipe->use);  // two host threads must not interleave their use of the events
    unsigned char* sA = cur;
    cur += round_up(e.a);
    unsigned char* sB = cur;
    cur += round_up(e.b);
    unsigned char* sR = cur;
    cur += round_up(e.r);
    unsigned char* sY = cur;
    if ((host_mask & COMFUSE_HOST_B)) {
      if (cudaMemcpyAsync(sB, B, e.b, cudaMemcpyHostToDevice, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
      dB = sB;
    }
    const bool host_r = (host_mask & COMFUSE_HOST_RESIDUAL) != 0;
    const unsigned char* hA = static_cast<const unsigned char*>(A);
    const unsigned char* hR = host_r ? static_cast<const unsigned char*>(args->residual) : nullptr;
    const unsigned char* dR = host_r ? sR : static_cast<const unsigned char*>(a.residual);
    unsigned char* hY = static_cast<unsigned char*>(Y);
    size_t ws_rows_bytes = 0;  // workspace bytes per row (dense Z of the unfused path, or the wide rows' partials)
    {
      size_t ws_all = 0;
      if (comfuse_workspace_size(desc, &ws_all) != COMFUSE_OK) return COMFUSE_ERR_INVALID_ARG;
      ws_rows_bytes = ws_all / static_cast<size_t>(desc->M);
      if (ws_all > 0 && (!workspace || workspace_bytes < ws_all)) return COMFUSE_ERR_WORKSPACE;
    }
    // from here on the helper streams are forked off the caller's stream: whatever happens, they are joined back
    // (`rejoin`), so that an error return leaves no work of this call outside the caller's stream order
    if (cudaEventRecord(pipe->fork, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    auto rejoin = [&](comfuse_status_t status) {
      const bool ok = cudaEventRecord(pipe->join, pipe->out) == cudaSuccess && cudaStreamWaitEvent(st, pipe->join, 0) == cudaSuccess &&
                      cudaEventRecord(pipe->join, pipe->in) == cudaSuccess && cudaStreamWaitEvent(st, pipe->join, 0) == cudaSuccess;
      return (status == COMFUSE_OK && !ok) ? COMFUSE_ERR_CUDA : status;
    };
    if (cudaStreamWaitEvent(pipe->in, pipe->fork, 0) != cudaSuccess) return rejoin(COMFUSE_ERR_CUDA);
    if (cudaStreamWaitEvent(pipe->out, pipe->fork, 0) != cudaSuccess) return rejoin(COMFUSE_ERR_CUDA);
    int c = 0;
    for (int r0 = 0; r0 < desc->M; r0 += rows_per_chunk, ++c) {
      const int rows = desc->M - r0 < rows_per_chunk ? desc->M - r0 : rows_per_chunk;
      const size_t offA = static_cast<size_t>(r0) * desc->lda * 2, offR = static_cast<size_t>(r0) * desc->ldr * 2,
                   offY = static_cast<size_t>(r0) * desc->ldy * 2;
      if (cudaMemcpyAsync(sA + offA, hA + offA, extent_bytes(1, rows, desc->K, desc->lda, 0), cudaMemcpyHostToDevice, pipe->in) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      if (host_r && cudaMemcpyAsync(sR + offR, hR + offR, extent_bytes(1, rows, desc->N, desc->ldr, 0), cudaMemcpyHostToDevice, pipe->in) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      if (cudaEventRecord(pipe->copied[c], pipe->in) != cudaSuccess || cudaStreamWaitEvent(st, pipe->copied[c], 0) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      comfuse_gemm_desc_t dc = *desc;
      dc.M = rows;
      comfuse_epilogue_args_t ac = a;
      if (dR) ac.residual = dR + offR;
      if (ac.row_max) ac.row_max += r0;
      if (ac.row_argmax) ac.row_argmax += r0;
      unsigned char* wsc = workspace ? static_cast<unsigned char*>(workspace) + static_cast<size_t>(r0) * ws_rows_bytes : nullptr;
      s = comfuse_gemm_epilogue(&dc, sA + offA, dB, sY + offY, &ac, wsc, wsc ? workspace_bytes - static_cast<size_t>(r0) * ws_rows_bytes : 0, cuda_stream);
      if (s != COMFUSE_OK) return rejoin(s);
      if (cudaEventRecord(pipe->computed[c], st) != cudaSuccess || cudaStreamWaitEvent(pipe->out, pipe->computed[c], 0) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      if (cudaMemcpyAsync(hY + offY, sY + offY, extent_bytes(1, rows, desc->N, desc->ldy, 0), cudaMemcpyDeviceToHost, pipe->out) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
    }
    return rejoin(COMFUSE_OK);
  }
  if ((host_mask & COMFUSE_HOST_A) && !stage_in(A, e.a, &dA)) return COMFUSE_ERR_CUDA;
  if ((host_mask & COMFUSE_HOST_B) && !stage_in(B, e.b, &dB)) return COMFUSE_ERR_CUDA;
  if ((host_mask & COMFUSE_HOST_RESIDUAL) && !stage_in(args->residual, e.r, &a.residual)) return COMFUSE_ERR_CUDA;
  if (host_mask & COMFUSE_HOST_Y) dY = cur;
  s = comfuse_gemm_epilogue(desc, dA, dB, dY, &a, workspace, workspace_bytes, cuda_stream);
  if (s != COMFUSE_OK) return s;
  if ((host_mask & COMFUSE_HOST_Y) && cudaMemcpyAsync(Y, dY, e.y, cudaMemcpyDeviceToHost, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  return COMFUSE_OK;
}

extern "C" comfuse_status_t comfuse_b2b_host_staging_size(const comfuse_b2b_desc_t* desc, size_t* bytes) {
  if (!desc || !bytes) return COMFUSE_ERR_INVALID_ARG;
  size_t ws = 0;
  const comfuse_status_t s = comfuse_b2b_workspace_size(desc, &ws);  // validates the description
  if (s != COMFUSE_OK) return s;
  const size_t nb = static_cast<size_t>(desc->batch);
  *bytes = round_up(nb * desc->M * desc->K * 2) + round_up(nb * desc->M * desc->N2 * 2);
  if (desc->kind == COMFUSE_B2B_SOFTMAX_ATTENTION)  // keys and values are per-step tensors too
    *bytes += round_up(nb * desc->K * desc->N1 * 2) + round_up(nb * desc->N1 * desc->N2 * 2);
  return COMFUSE_OK;
}

extern "C" comfuse_status_t comfuse_b2b_gemm_host(const comfuse_b2b_desc_t* desc, const void* X, const void* W1, const void* b1,
                                                  const void* W2, const void* b2, const void* gamma, const void* beta, void* O,
                                                  void* staging, size_t staging_bytes, void* workspace,
                                                  size_t workspace_bytes, void* cuda_stream) {
  size_t need = 0;
  comfuse_status_t s = comfuse_b2b_host_staging_size(desc, &need);
  if (s != COMFUSE_OK) return s;
  if (!X || !O) return COMFUSE_ERR_INVALID_ARG;
  if (!staging || staging_bytes < need) return COMFUSE_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(staging) & 15u) return COMFUSE_ERR_ALIGNMENT;
  {  // everything that can be checked on the host is checked before the first copy is enqueued
    size_t ws_all = 0;
    if (comfuse_b2b_workspace_size(desc, &ws_all) != COMFUSE_OK) return COMFUSE_ERR_INVALID_ARG;
    if (ws_all > 0 && (!workspace || workspace_bytes < ws_all)) return COMFUSE_ERR_WORKSPACE;
    if (ws_all > 0 && (reinterpret_cast<uintptr_t>(workspace) & 15u)) return COMFUSE_ERR_ALIGNMENT;
    if (!W1 || !W2) return COMFUSE_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t nb = static_cast<size_t>(desc->batch);
  const size_t xb = nb * desc->M * desc->K * 2, ob = nb * desc->M * desc->N2 * 2;
  unsigned char* dX = static_cast<unsigned char*>(staging);
  unsigned char* dO = dX + round_up(xb);
  // ---- pipelined form: row ranges (MLP kind) or batch ranges (attention kind) flow through copy-in, compute and copy-out
  // streams like the GEMM form above
  const bool attn = desc->kind == COMFUSE_B2B_SOFTMAX_ATTENTION;
  const long long units = attn ? desc->batch : desc->M;                     // what is cut: batches or rows
  const long long grain = attn ? 1 : 256;
  const int nchunks = pipe_chunks(xb + (attn ? nb * (static_cast<size_t>(desc->K) * desc->N1 + static_cast<size_t>(desc->N1) * desc->N2) * 2 : 0));
  const long long per_chunk = nchunks >= 2 ? ((units + nchunks - 1) / nchunks + grain - 1) / grain * grain : units;
  Pipe* pipe = (nchunks >= 2 && units >= 2 * per_chunk && (!attn || (W1 && W2))) ? pipe_for_current_device() : nullptr;
  if (pipe) {
    std::lock_guard<std::mutex> one_call(pipe->use);  // two host threads must not interleave their use of the events
    const size_t w1b = nb * desc->K * desc->N1 * 2, w2b = nb * desc->N1 * desc->N2 * 2;
    unsigned char* dW1 = dO + round_up(ob);
    unsigned char* dW2 = dW1 + round_up(w1b);
    size_t ws_all = 0;
    if (comfuse_b2b_workspace_size(desc, &ws_all) != COMFUSE_OK) return COMFUSE_ERR_INVALID_ARG;
    if (ws_all > 0 && (!workspace || workspace_bytes < ws_all)) return COMFUSE_ERR_WORKSPACE;
    const size_t ws_unit = ws_all / static_cast<size_t>(units);
    // bytes per unit (row or batch) of each per-step tensor
    const size_t ux = static_cast<size_t>(attn ? desc->M : 1) * desc->K * 2, uo = static_cast<size_t>(attn ? desc->M : 1) * desc->N2 * 2;
    const size_t u1 = static_cast<size_t>(desc->K) * desc->N1 * 2, u2 = static_cast<size_t>(desc->N1) * desc->N2 * 2;
    if (cudaEventRecord(pipe->fork, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    auto rejoin = [&](comfuse_status_t status) {  // whatever happens, the helper streams are joined back into the caller's
      const bool ok = cudaEventRecord(pipe->join, pipe->out) == cudaSuccess && cudaStreamWaitEvent(st, pipe->join, 0) == cudaSuccess &&
                      cudaEventRecord(pipe->join, pipe->in) == cudaSuccess && cudaStreamWaitEvent(st, pipe->join, 0) == cudaSuccess;
      return (status == COMFUSE_OK && !ok) ? COMFUSE_ERR_CUDA : status;
    };
    if (cudaStreamWaitEvent(pipe->in, pipe->fork, 0) != cudaSuccess || cudaStreamWaitEvent(pipe->out, pipe->fork, 0) != cudaSuccess)
      return rejoin(COMFUSE_ERR_CUDA);
    int c = 0;
    for (long long u0 = 0; u0 < units; u0 += per_chunk, ++c) {
      const long long n = units - u0 < per_chunk ? units - u0 : per_chunk;
      const unsigned char* hX = static_cast<const unsigned char*>(X) + u0 * ux;
      if (cudaMemcpyAsync(dX + u0 * ux, hX, n * ux, cudaMemcpyHostToDevice, pipe->in) != cudaSuccess) return rejoin(COMFUSE_ERR_CUDA);
      if (attn) {
        if (cudaMemcpyAsync(dW1 + u0 * u1, static_cast<const unsigned char*>(W1) + u0 * u1, n * u1, cudaMemcpyHostToDevice, pipe->in) != cudaSuccess ||
            cudaMemcpyAsync(dW2 + u0 * u2, static_cast<const unsigned char*>(W2) + u0 * u2, n * u2, cudaMemcpyHostToDevice, pipe->in) != cudaSuccess)
          return rejoin(COMFUSE_ERR_CUDA);
      }
      if (cudaEventRecord(pipe->copied[c], pipe->in) != cudaSuccess || cudaStreamWaitEvent(st, pipe->copied[c], 0) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      comfuse_b2b_desc_t dc = *desc;
      if (attn) dc.batch = static_cast<int32_t>(n);
      else dc.M = static_cast<int32_t>(n);
      unsigned char* wsc = workspace ? static_cast<unsigned char*>(workspace) + u0 * ws_unit : nullptr;
      s = comfuse_b2b_gemm(&dc, dX + u0 * ux, attn ? static_cast<const void*>(dW1 + u0 * u1) : W1, b1,
                           attn ? static_cast<const void*>(dW2 + u0 * u2) : W2, b2, gamma, beta, dO + u0 * uo, wsc,
                           wsc ? workspace_bytes - u0 * ws_unit : 0, cuda_stream);
      if (s != COMFUSE_OK) return rejoin(s);
      if (cudaEventRecord(pipe->computed[c], st) != cudaSuccess || cudaStreamWaitEvent(pipe->out, pipe->computed[c], 0) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
      if (cudaMemcpyAsync(static_cast<unsigned char*>(O) + u0 * uo, dO + u0 * uo, n * uo, cudaMemcpyDeviceToHost, pipe->out) != cudaSuccess)
        return rejoin(COMFUSE_ERR_CUDA);
    }
    return rejoin(COMFUSE_OK);
  }
  if (cudaMemcpyAsync(dX, X, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  if (desc->kind == COMFUSE_B2B_SOFTMAX_ATTENTION) {  // W1 (keys) and W2 (values) are host pointers as well
    if (!W1 || !W2) return COMFUSE_ERR_INVALID_ARG;
    const size_t w1b = nb * desc->K * desc->N1 * 2, w2b = nb * desc->N1 * desc->N2 * 2;
    unsigned char* dW1 = dO + round_up(ob);
    unsigned char* dW2 = dW1 + round_up(w1b);
    if (cudaMemcpyAsync(dW1, W1, w1b, cudaMemcpyHostToDevice, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    if (cudaMemcpyAsync(dW2, W2, w2b, cudaMemcpyHostToDevice, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
    W1 = dW1;
    W2 = dW2;
  }
  s = comfuse_b2b_gemm(desc, dX, W1, b1, W2, b2, gamma, beta, dO, workspace, workspace_bytes, cuda_stream);
  if (s != COMFUSE_OK) return s;
  if (cudaMemcpyAsync(O, dO, ob, cudaMemcpyDeviceToHost, st) != cudaSuccess) return COMFUSE_ERR_CUDA;
  return COMFUSE_OK;
}
