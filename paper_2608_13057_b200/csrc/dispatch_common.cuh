// Pieces shared by the two count+dispatch kernels (quota and sampled).
#pragma once

#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kDispThreads = 1024;
constexpr int kDispWarps = kDispThreads / 32;
constexpr int kKeep = 4;           // 32-pair steps of a warp whose ids stay in registers between the passes
constexpr int kMaxCluster = 16;    // largest cluster on this part (beyond 8 is opt-in per kernel; checked per device)
constexpr int kPairsPerCta = 1024;
constexpr int kMaxShare = 1 << 30;   // largest share x_{e,r} the quota dispatch accepts
constexpr size_t kDispatchSmemLimit = 220 * 1024;   // the shape check rejects tables beyond this // pairs per CTA before another CTA joins the cluster

// Lanes of the warp that hold the same expert id as this lane (e < 0: none).  One ballot per id
// bit: a fixed, short latency, where __match_any_sync takes one round per distinct value.
__device__ __forceinline__ uint32_t same_expert_mask(int e, int id_bits) {
  uint32_t m = __ballot_sync(0xffffffffu, e >= 0);
  for (int b = 0; b < id_bits; ++b) {
    const uint32_t bal = __ballot_sync(0xffffffffu, (e >> b) & 1);
    m &= ((e >> b) & 1) ? bal : ~bal;
  }
  return e >= 0 ? m : 0u;
}

// Exclusive scan of 128*ceil(m/128) over the G instance slots in ascending slot id, by warp 0:
// off[0..G], off[G] = padded rows in use.  Call with all threads of warp 0; s_carry is one shared int.
__device__ __forceinline__ void padded_offsets_warp0(const int32_t* m_inst, int32_t* off, int G, int lane, int32_t* s_carry) {
  if (lane == 0) *s_carry = 0;
  __syncwarp();
  for (int base = 0; base < G; base += 32) {
    const int i = base + lane;
    const int padded = i < G ? ((m_inst[i] + kTileM - 1) / kTileM) * kTileM : 0;
    int incl = padded;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    const int carry = *s_carry;
    if (i < G) off[i] = carry + incl - padded;
    __syncwarp();
    if (lane == 31) *s_carry = carry + incl;
    __syncwarp();
  }
  if (lane == 0) off[G] = *s_carry;
}

// First i with off[i+1] > row (the instance owning a row below off[G]).
__device__ __forceinline__ int instance_of_row(const int32_t* off, int G, int row) {
  int lo = 0, hi = G;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (off[mid + 1] > row) hi = mid; else lo = mid + 1;
  }
  return lo;
}

inline int dispatch_cluster_size(long long pairs, int max_cluster) {
  int nc = 1;
  while (nc < max_cluster && static_cast<long long>(nc) * kPairsPerCta < pairs) nc *= 2;
  return nc;
}

// Largest cluster the kernel can run on the current device: 16 where the device can place a cluster of 16
// such CTAs in one GPC (asked once per device), else the portable 8.
template <typename Params>
inline int dispatch_max_cluster(void (*kernel)(Params), size_t smem) {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 8;
  const int have = cached[dev].load(std::memory_order_acquire);
  if (have != 0) return have;
  int best = 8;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kMaxCluster);
    cfg.blockDim = dim3(kDispThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kMaxCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n > 0) best = kMaxCluster;
    else (void)cudaGetLastError();                 // a refused query must not poison the next launch
  } else {
    (void)cudaGetLastError();
  }
  cached[dev].store(best, std::memory_order_release);
  return best;
}

template <typename Params>
inline cudaError_t launch_dispatch_cluster(void (*kernel)(Params), const Params& p, long long pairs, size_t smem,
                                           cudaStream_t stream) {
  // (the limit is raised to the largest table the shape checks admit, once per device and kernel)
  static std::atomic<unsigned long long> smem_set{0};
  cudaError_t e = smem_limit_once(kernel, kDispatchSmemLimit, smem_set);
  if (e != cudaSuccess) return e;
  const int nc = dispatch_cluster_size(pairs, dispatch_max_cluster(kernel, kDispatchSmemLimit));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(nc);
  cfg.blockDim = dim3(kDispThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = nc;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

}  // namespace tempo
