// Host-side launch of the short-K row-softmax kernel (pairs of CTAs, persistent grid).
#include <atomic>
#include <cstdio>
#include <cstdlib>

#include "host_common.h"
#include "softmax_rows.cuh"

namespace comfuse {

bool softmax_rows_supported(const FusedParams& p) { return p.K <= 256 && p.N >= 64; }

cudaError_t launch_softmax_rows(const GemmMaps& maps, FusedParams p, cudaStream_t stream) {
  constexpr int NSTAGES = 2, YBOXES = 2;
  using Cfg = RowSoftmaxCfg<NSTAGES, YBOXES>;
  auto kern = p.b_nk ? softmax_rows_kernel<NSTAGES, YBOXES, true> : softmax_rows_kernel<NSTAGES, YBOXES, false>;
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  constexpr int kMaxDev = 64;
  static std::atomic<int> max_clusters[kMaxDev];  // 0 = kernel not configured yet on that device (set last, released)
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;

  p.mpairs = (p.mblocks + 1) / 2;
  p.nblocks = 1;
  p.total_tiles = p.batch * p.mpairs;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic_launch_enabled() ? 2 : 1;

  int ncl = max_clusters[di].load(std::memory_order_acquire);
  if (ncl == 0) {
    cudaError_t e = cudaFuncSetAttribute(softmax_rows_kernel<NSTAGES, YBOXES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(softmax_rows_kernel<NSTAGES, YBOXES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    int n = 0;
    cfg.gridDim = dim3(2 * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
    if (std::getenv("COMFUSE_VERBOSE"))
      std::fprintf(stderr, "comfuse: row-softmax kernel: %d pairs fit, %d B smem\n", n, Cfg::SMEM_BYTES);
  }
  const int clusters = p.total_tiles < ncl ? p.total_tiles : ncl;
  if (clusters <= 0) return cudaSuccess;
  cfg.gridDim = dim3(clusters * 2, 1, 1);
  count_launch();
  return cudaLaunchKernelEx(&cfg, kern, maps.A, maps.B, maps.Y, p);
}

}  // namespace comfuse
