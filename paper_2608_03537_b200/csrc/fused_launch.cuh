// Host-side launch of one fused_pair_kernel instantiation: shared-memory opt-in, cluster dimensions (2*CN CTAs,
// non-portable size when above 8), persistent grid sized from the number of clusters the device can hold at once.
#pragma once

#include <atomic>
#include <cstdio>
#include <cstdlib>

#include "fused_pair.cuh"
#include "host_common.h"

namespace comfuse {

// What a launch needs to know about one instantiation of the kernel.
struct PairLaunchShape {
  int threads, smem_bytes, cluster;
};
constexpr int kMaxLaunchDevices = 64;

// One work item = a pair of adjacent 128-row blocks (times p.nblocks column blocks of CN*BN columns).  `kern` is a
// __global__ function of this library or a kernel handle of a module compiled at run time; `max_clusters` caches, per
// device, how many clusters of it fit at once (0 = not configured yet on that device; set last, released).
inline cudaError_t launch_pair_kernel(const void* kern, std::atomic<int>* max_clusters, const PairLaunchShape& sh, const char* what,
                                      const GemmMaps& maps, FusedParams p, cudaStream_t stream) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  const int di = dev->device < kMaxLaunchDevices ? dev->device : kMaxLaunchDevices - 1;

  p.mpairs = (p.mblocks + 1) / 2;
  if (p.nblocks < 1) p.nblocks = 1;
  p.total_tiles = p.batch * p.mpairs * p.nblocks;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(sh.threads, 1, 1);
  cfg.dynamicSmemBytes = sh.smem_bytes;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = sh.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic_launch_enabled() ? 2 : 1;

  int ncl = max_clusters[di].load(std::memory_order_acquire);
  if (ncl == 0) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sh.smem_bytes);
    if (e != cudaSuccess) return e;
    if (sh.cluster > 8) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
    }
    int n = 0;
    cfg.gridDim = dim3(sh.cluster * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
    if (std::getenv("COMFUSE_VERBOSE"))
      std::fprintf(stderr, "comfuse: kernel %s: cluster of %d CTAs, %d clusters fit, %d B smem\n", what, sh.cluster, n, sh.smem_bytes);
  }
  const int clusters = p.total_tiles < ncl ? p.total_tiles : ncl;
  if (clusters <= 0) return cudaSuccess;
  cfg.gridDim = dim3(clusters * sh.cluster, 1, 1);
  count_launch();
  void* args[5] = {const_cast<CUtensorMap*>(&maps.A), const_cast<CUtensorMap*>(&maps.B), const_cast<CUtensorMap*>(&maps.R),
                   const_cast<CUtensorMap*>(&maps.Y), &p};
  return cudaLaunchKernelExC(&cfg, kern, args);
}

template <int EPI, int BNS0, int BNS1, int CN, int NSTAGES, int LOCK = 0, int EPW = 2>
cudaError_t launch_pair_instance(const GemmMaps& maps, const FusedParams& p, cudaStream_t stream) {
  using Cfg = PairCfg<EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW>;
  static std::atomic<int> max_clusters[kMaxLaunchDevices];
  char what[96];
  std::snprintf(what, sizeof(what), "epi=%d bns=%d+%d cn=%d stages=%d lock=%d epw=%d, %d staging boxes/warp", EPI, BNS0, BNS1, CN, NSTAGES, LOCK,
                EPW, Cfg::YBOXES);
  return launch_pair_kernel(reinterpret_cast<const void*>(&fused_pair_kernel<EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW>), max_clusters,
                            PairLaunchShape{Cfg::kThreads, Cfg::SMEM_BYTES, 2 * CN}, what, maps, p, stream);
}

// The stage-program instantiations (tile widths, cluster size, pipeline depth, lock-step) by row length N:
// X(N, BNS0, BNS1, CN, NSTAGES, LOCK).  One table for the interpreter's instantiations and for the kernels compiled at run time.
#define COMFUSE_PROGRAM_INSTANCES_SMALL(X) X(256, 256, 0, 1, 5, 0) X(512, 256, 256, 1, 3, 1) X(768, 256, 128, 2, 4, 1)
#define COMFUSE_PROGRAM_INSTANCES_LARGE(X) X(1024, 256, 256, 2, 3, 1) X(2048, 256, 256, 4, 3, 1) X(4096, 256, 256, 8, 3, 1)
// Further row lengths for the kernels generated at run time (an instantiation there costs a table entry, not a translation
// unit): clusters of 6, 10, 12 and 14 CTAs.
#define COMFUSE_PROGRAM_INSTANCES_GENERATED_ONLY(X) \
  X(1280, 256, 0, 5, 5, 0) X(1536, 256, 256, 3, 3, 1) X(1792, 256, 0, 7, 5, 0) X(2560, 256, 256, 5, 3, 1) X(3072, 256, 256, 6, 3, 1) \
  X(3584, 256, 256, 7, 3, 1)

}  // namespace comfuse
