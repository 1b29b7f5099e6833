// Host-buffer forms of the two entry points: the per-step tensors (activations in, result out) are HOST pointers; the
// call copies them to / from a device staging area the caller provides and runs the same kernels in between, all on the
// caller's stream.  Nothing is allocated; the staging layout keeps the tensors' own strides, so every copy is one
// contiguous cudaMemcpyAsync of the tensor's extent.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/comfuse.h"

namespace {

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
  if (mask & COMFUSE_HOST_B) e.b = extent_bytes(d->batch, d->K, d->N, d->ldb, d->batch_stride_b);
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
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t nb = static_cast<size_t>(desc->batch);
  const size_t xb = nb * desc->M * desc->K * 2, ob = nb * desc->M * desc->N2 * 2;
  unsigned char* dX = static_cast<unsigned char*>(staging);
  unsigned char* dO = dX + round_up(xb);
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
