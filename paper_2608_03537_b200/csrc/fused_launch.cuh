// Host-side launch of one fused_pair_kernel instantiation: shared-memory opt-in, cluster dimensions (2*CN CTAs,
// non-portable size when above 8), persistent grid sized from the number of clusters the device can hold at once.
#pragma once

#include <atomic>
#include <cstdio>
#include <cstdlib>

#include "fused_pair.cuh"
#include "host_common.h"

namespace comfuse {

// One work item = a pair of adjacent 128-row blocks (times p.nblocks column blocks of CN*BN columns).
template <int EPI, int BNS0, int BNS1, int CN, int NSTAGES, int LOCK = 0, int EPW = 2>
cudaError_t launch_pair_instance(const GemmMaps& maps, FusedParams p, cudaStream_t stream) {
  using Cfg = PairCfg<EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW>;
  auto kern = fused_pair_kernel<EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW>;
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  constexpr int kCluster = 2 * CN;
  constexpr int kMaxDev = 64;
  static std::atomic<int> max_clusters[kMaxDev];  // 0 = kernel not configured yet on that device (set last, released)
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;

  p.mpairs = (p.mblocks + 1) / 2;
  if (p.nblocks < 1) p.nblocks = 1;
  p.total_tiles = p.batch * p.mpairs * p.nblocks;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic_launch_enabled() ? 2 : 1;

  int ncl = max_clusters[di].load(std::memory_order_acquire);
  if (ncl == 0) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if (kCluster > 8) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
    }
    int n = 0;
    cfg.gridDim = dim3(kCluster * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
    if (std::getenv("COMFUSE_VERBOSE"))
      std::fprintf(stderr, "comfuse: kernel epi=%d bns=%d+%d cn=%d stages=%d lock=%d epw=%d: cluster of %d CTAs, %d clusters fit, %d B smem, %d staging boxes/warp\n",
                   EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW, kCluster, n, Cfg::SMEM_BYTES, Cfg::YBOXES);
  }
  const int clusters = p.total_tiles < ncl ? p.total_tiles : ncl;
  if (clusters <= 0) return cudaSuccess;
  cfg.gridDim = dim3(clusters * kCluster, 1, 1);
  count_launch();
  return cudaLaunchKernelEx(&cfg, kern, maps.A, maps.B, maps.R, maps.Y, p);
}

}  // namespace comfuse
