// Step 4: weighted un-permute.  out[t,:] = sum over the token's k slots, in slot order, of
// topk_w[t,s] * y[pair_row[t,s],:] with fp32 accumulation and a bf16 store (the "combine" of
// Section 2.1 restricted to this rank's partial sum).  HBM-bound gather: one CTA per token,
// 16-byte loads and stores.
#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kCombThreads = 128;
constexpr int kMaxK = 32;


__global__ void __launch_bounds__(kCombThreads) combine_kernel(const CombineParams p) {
  __shared__ int32_t s_row[kMaxK];
  __shared__ float s_w[kMaxK];
  const int t = blockIdx.x;
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));
  if (threadIdx.x < p.k) {
    const int idx = t * p.k + threadIdx.x;
    s_row[threadIdx.x] = t < nv ? p.pair_row[idx] : -1;
    s_w[threadIdx.x] = p.topk_w[idx];
  }
  __syncthreads();
  __nv_bfloat16* dst = p.out + static_cast<size_t>(t) * p.d;
  for (int col = threadIdx.x * 8; col < p.d; col += kCombThreads * 8) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < p.k; ++s) {
      const int row = s_row[s];
      if (row < 0) continue;
      const float w = s_w[s];
      const uint4 v = *reinterpret_cast<const uint4*>(p.y + static_cast<size_t>(row) * p.d + col);
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
        acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
      }
    }
    uint4 o;
    uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
      ou[i] = *reinterpret_cast<const uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(dst + col) = o;
  }
}

cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream) {
  combine_kernel<<<p.T, kCombThreads, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace tempo
