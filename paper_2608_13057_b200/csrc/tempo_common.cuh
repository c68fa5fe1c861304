// Shared device helpers of the expert-block kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "tempo.h"

namespace tempo {

constexpr int kTileM = 128;     // rows per M-tile (Eq. 3)
constexpr int kQBlock = 128;    // columns per activation scale

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Index of the scale byte of (row, column block kb) in the 512-byte atom layout (see tempo.h).
__device__ __forceinline__ size_t sf_index(int row, int kb, int J) {
  return (static_cast<size_t>(row >> 7) * J + (kb >> 2)) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4 + (kb & 3);
}

// Smallest integer eps with amax <= 448 * 2^eps (0 if amax == 0), clamped to [-126, 127], from the
// bits of amax: amax = m * 2^L with m in [1,2) and 448 = 1.75 * 2^8.
__device__ __forceinline__ int pow2_scale_exponent(float amax) {
  const uint32_t bits = __float_as_uint(amax) & 0x7fffffffu;
  if (bits == 0) return 0;
  const int ef = static_cast<int>(bits >> 23);
  if (ef == 0) return -126;                       // denormal maximum
  int eps = ef - 127 - 8 + ((bits & 0x7fffffu) > 0x600000u ? 1 : 0);
  return max(-126, min(127, eps));
}

// 2^(-eps) for eps in [-126, 127].
__device__ __forceinline__ float pow2_neg(int eps) {
  return eps <= 126 ? __uint_as_float(static_cast<uint32_t>(127 - eps) << 23) : __uint_as_float(0x00400000u);
}

// Two floats -> two e4m3 codes (round to nearest even, saturating), lo in bits [0,8).
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ uint32_t cvt_e4m3x4(float a, float b, float c, float d) {
  return cvt_e4m3x2(a, b) | (cvt_e4m3x2(c, d) << 16);
}

// Programmatic dependent launch: every hot-path kernel lets its successor in the stream start
// launching at once (pdl_trigger) and itself touches global memory only after its predecessor has
// completed and flushed (pdl_wait), so launch latency and kernel prologues overlap the previous
// kernel's tail.  Both are no-ops when the kernel was launched without the attribute.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Default bound of the device-side waits of the FFN kernel (tempo_grouped_ffn_bounded takes another).
constexpr unsigned long long kDefaultWaitNs = 50ull * 1000ull * 1000ull;

// Raises a kernel's dynamic shared-memory limit once per device and kernel instead of on every launch.
// `done` is a bit mask over device ordinals owned by the caller (one static per kernel); a race between
// two first calls sets the attribute twice, which is harmless.
template <typename Kernel>
inline cudaError_t smem_limit_once(Kernel kernel, size_t bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
  if (bit != 0 && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
  if (e == cudaSuccess && bit != 0) done.fetch_or(bit, std::memory_order_release);
  return e;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace tempo
