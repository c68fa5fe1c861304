// Step 4: weighted un-permute.  out[t,:] = sum over the token's k slots, in slot order, of
// topk_w[t,s] * y[pair_row[t,s],:] with fp32 accumulation and a bf16 store (the "combine" of
// Section 2.1 restricted to this rank's partial sum).  HBM-bound gather with
// 16-byte loads and stores.
#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kCombThreads = 256;
constexpr int kGroup = 4;   // slots whose gathers are in flight together

// One thread per (token, 8 columns).  The k row indices and weights are read first, then all
// gathers of a group of kGroup slots are issued before any is consumed, so the thread pays the memory
// latency once per group instead of once per slot; the sum itself stays in slot order.
__global__ void __launch_bounds__(kCombThreads, 6) combine_kernel(const CombineParams p) {
  const int t = blockIdx.x;
  const int col = (blockIdx.y * kCombThreads + threadIdx.x) * 8;
  pdl_trigger();
  if (col >= p.d) return;
  pdl_wait();
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (t < nv) {
    for (int s0 = 0; s0 < p.k; s0 += kGroup) {
      int row[kGroup];
      float w[kGroup];
      uint4 v[kGroup];
#pragma unroll
      for (int i = 0; i < kGroup; ++i) {
        const int s = s0 + i;
        row[i] = s < p.k ? __ldg(p.pair_row + t * p.k + s) : -1;
        w[i] = s < p.k ? __ldg(p.topk_w + t * p.k + s) : 0.f;
      }
#pragma unroll
      for (int i = 0; i < kGroup; ++i)
        v[i] = row[i] >= 0 ? __ldcs(reinterpret_cast<const uint4*>(p.y + static_cast<size_t>(row[i]) * p.d + col))
                           : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int i = 0; i < kGroup; ++i) {
        if (row[i] < 0) continue;
        const uint32_t u[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] = fmaf(w[i], __uint_as_float(u[j] << 16), acc[2 * j]);
          acc[2 * j + 1] = fmaf(w[i], __uint_as_float(u[j] & 0xffff0000u), acc[2 * j + 1]);
        }
      }
    }
  }
  uint4 o;
  uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    ou[i] = *reinterpret_cast<const uint32_t*>(&b);
  }
  __stcs(reinterpret_cast<uint4*>(p.out + static_cast<size_t>(t) * p.d + col), o);
}

cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream) {
  const dim3 grid(p.T, (p.d / 8 + kCombThreads - 1) / kCombThreads);
  return launch_pdl(combine_kernel, grid, dim3(kCombThreads), 0, stream, p);
}

}  // namespace tempo
