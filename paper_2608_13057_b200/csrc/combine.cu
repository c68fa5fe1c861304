// Step 4: weighted un-permute.  out[t,:] = sum over the token's k slots, in slot order, of
// topk_w[t,s] * y[pair_row[t,s],:] with fp32 accumulation and a bf16 store (the "combine" of
// Section 2.1 restricted to this rank's partial sum).  HBM-bound gather with
// 16-byte loads and stores.
#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kCombThreads = 256;

// One thread per (N consecutive tokens, 8 columns).  The row indices and weights of a group of GROUP
// slots are read first for every token, then all their gathers are issued before any is consumed, so
// the thread pays the memory latency once per group instead of once per slot; each token's sum stays
// in slot order.  N * GROUP gathers of 16 bytes are in flight per thread: with few slots per token
// (small k) N is raised so that an SM still keeps enough bytes in flight to cover the HBM latency.
template <int N, int GROUP>
__global__ void __launch_bounds__(kCombThreads, N == 1 ? 6 : 4) combine_kernel(const CombineParams p) {
  const int t0 = blockIdx.x * N;
  const int col = (blockIdx.y * kCombThreads + threadIdx.x) * 8;
  pdl_trigger();
  if (col >= p.d) return;
  pdl_wait();
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));
  float acc[N][8];
#pragma unroll
  for (int n = 0; n < N; ++n)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[n][j] = 0.f;
  for (int s0 = 0; s0 < p.k; s0 += GROUP) {
    int row[N][GROUP];
    float w[N][GROUP];
    uint4 v[N][GROUP];
#pragma unroll
    for (int n = 0; n < N; ++n)
#pragma unroll
      for (int i = 0; i < GROUP; ++i) {
        const int s = s0 + i;
        const bool on = s < p.k && t0 + n < nv;
        row[n][i] = on ? __ldg(p.pair_row + (t0 + n) * p.k + s) : -1;
        w[n][i] = on ? __ldg(p.topk_w + (t0 + n) * p.k + s) : 0.f;
      }
#pragma unroll
    for (int n = 0; n < N; ++n)
#pragma unroll
      for (int i = 0; i < GROUP; ++i)
        v[n][i] = row[n][i] >= 0 ? __ldcs(reinterpret_cast<const uint4*>(p.y + static_cast<size_t>(row[n][i]) * p.d + col))
                                 : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int n = 0; n < N; ++n)
#pragma unroll
      for (int i = 0; i < GROUP; ++i) {
        if (row[n][i] < 0) continue;
        const uint32_t u[4] = {v[n][i].x, v[n][i].y, v[n][i].z, v[n][i].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[n][2 * j] = fmaf(w[n][i], __uint_as_float(u[j] << 16), acc[n][2 * j]);
          acc[n][2 * j + 1] = fmaf(w[n][i], __uint_as_float(u[j] & 0xffff0000u), acc[n][2 * j + 1]);
        }
      }
  }
#pragma unroll
  for (int n = 0; n < N; ++n) {
    if (t0 + n >= p.T) break;
    uint4 o;
    uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 b = __floats2bfloat162_rn(acc[n][2 * i], acc[n][2 * i + 1]);
      ou[i] = *reinterpret_cast<const uint32_t*>(&b);
    }
    __stcs(reinterpret_cast<uint4*>(p.out + static_cast<size_t>(t0 + n) * p.d + col), o);
  }
}

template <int N, int GROUP>
static cudaError_t launch_combine_t(const CombineParams& p, cudaStream_t stream) {
  const dim3 grid((p.T + N - 1) / N, (p.d / 8 + kCombThreads - 1) / kCombThreads);
  return launch_pdl(combine_kernel<N, GROUP>, grid, dim3(kCombThreads), 0, stream, p);
}

cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream) {
  if (p.k <= 1) return launch_combine_t<4, 1>(p, stream);
  if (p.k <= 2) return launch_combine_t<2, 2>(p, stream);
  return launch_combine_t<1, 4>(p, stream);
}

}  // namespace tempo
