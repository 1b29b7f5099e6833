// Host-side launch of one fused_gemm_kernel instantiation: shared-memory opt-in, cluster dimensions,
// persistent grid sized from the number of clusters the device can hold at once.
#pragma once

#include "fused_gemm.cuh"
#include "fused_pair.cuh"
#include "host_common.h"

namespace comfuse {

template <int EPI, int BNS, int NSUB, int CN, int NSTAGES>
cudaError_t launch_fused_instance(const CUtensorMap& tmA, const CUtensorMap& tmB, const FusedParams& p, cudaStream_t stream) {
  using Cfg = FusedCfg<EPI, BNS, NSUB, CN, NSTAGES>;
  auto kern = fused_gemm_kernel<EPI, BNS, NSUB, CN, NSTAGES>;
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;

  constexpr int kMaxDev = 64;
  static int max_clusters[kMaxDev] = {0};  // 0 = not configured yet on that device
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  if (CN > 1) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CN;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.numAttrs = 1;
  }

  if (max_clusters[di] == 0) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    int n = 0;
    if (CN > 1) {
      cfg.gridDim = dim3(CN * dev->sm_count, 1, 1);
      e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
      if (e != cudaSuccess) return e;
    } else {
      n = dev->sm_count;  // one CTA per SM (shared memory and TMEM both allow only one)
    }
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di] = n;
  }
  const int clusters = p.total_tiles < max_clusters[di] ? p.total_tiles : max_clusters[di];
  if (clusters <= 0) return cudaSuccess;
  cfg.gridDim = dim3(clusters * CN, 1, 1);
  count_launch();
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, p);
}

// CTA-pair kernels: clusters of 2*CN CTAs, one work item = a pair of adjacent row blocks (times nblocks column blocks).
template <int EPI, int BNS0, int BNS1, int CN, int NACC, int NSTAGES>
cudaError_t launch_pair_instance(const CUtensorMap& tmA, const CUtensorMap& tmB, FusedParams p, cudaStream_t stream) {
  using Cfg = PairCfg<EPI, BNS0, BNS1, CN, NACC, NSTAGES>;
  auto kern = fused_pair_kernel<EPI, BNS0, BNS1, CN, NACC, NSTAGES>;
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  constexpr int kCluster = 2 * CN;
  constexpr int kMaxDev = 64;
  static int max_clusters[kMaxDev] = {0};
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;

  p.mpairs = (p.mblocks + 1) / 2;
  if (p.nblocks < 1) p.nblocks = 1;
  p.total_tiles = p.batch * p.mpairs * p.nblocks;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  cfg.blockDim = dim3(Cfg::kThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;

  if (max_clusters[di] == 0) {
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
    max_clusters[di] = n;
  }
  const int clusters = p.total_tiles < max_clusters[di] ? p.total_tiles : max_clusters[di];
  if (clusters <= 0) return cudaSuccess;
  cfg.gridDim = dim3(clusters * kCluster, 1, 1);
  count_launch();
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, p);
}

}  // namespace comfuse
