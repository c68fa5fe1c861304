// Step 2: gather token rows into the padded grouped layout and quantise them to fp8 e4m3 with one
// power-of-two scale per 128 columns (the "scatter/gather, quantization" per-token kernels of the
// paper's full-pipeline scope, Appendix B).  HBM-bound: one warp per row, 32-byte loads per lane,
// 16-byte stores; the block maximum is reduced over the 8 lanes that share a 128-column block.
#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kPermWarps = 8;


// One warp per (row, 512-column chunk), grid-stride over the rows in use, two items per trip so the
// gathers of both are in flight together: a lane loads 32 bytes, the 8 lanes of a 128-column block
// reduce its maximum, every lane stores 16 code bytes.
struct PermItem {
  int row, col, pair;
  bool live, in;
  uint4 lo, hi;
};

__device__ __forceinline__ void perm_load(const PermuteParams& p, int row, int chunk, bool live, int lane, PermItem& it) {
  it.live = live;
  it.row = live ? row : 0;
  it.col = live ? chunk * 512 + lane * 16 : 0;
  it.in = live && it.col < p.d;                     // d is a multiple of 128, so 8-lane groups agree
  it.pair = live ? __ldg(p.row_pair + it.row) : -1;
  it.lo = make_uint4(0, 0, 0, 0);
  it.hi = make_uint4(0, 0, 0, 0);
}

__device__ __forceinline__ void perm_gather(const PermuteParams& p, PermItem& it) {
  if (it.in && it.pair >= 0) {
    const __nv_bfloat16* src = p.x + static_cast<size_t>(it.pair / p.k) * p.d + it.col;
    it.lo = __ldcs(reinterpret_cast<const uint4*>(src));
    it.hi = __ldcs(reinterpret_cast<const uint4*>(src + 8));
  }
}

__device__ __forceinline__ void perm_finish(const PermuteParams& p, const PermItem& it, int lane, int J) {
  // padding rows come out as zero codes with scale 1 (all-zero block: eps = 0)
  const uint32_t w[8] = {it.lo.x, it.lo.y, it.lo.z, it.lo.w, it.hi.x, it.hi.y, it.hi.z, it.hi.w};
  // block maximum on the packed bf16 pairs (magnitudes compare like the floats they stand for)
  __nv_bfloat162 m2 = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[0]));
#pragma unroll
  for (int i = 1; i < 8; ++i) m2 = __hmax2(m2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
  const uint32_t mbits = *reinterpret_cast<const uint32_t*>(&m2);
  float amax = fmaxf(__uint_as_float(mbits << 16), __uint_as_float(mbits & 0xffff0000u));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
  if (!it.in) return;
  const int eps = pow2_scale_exponent(amax);
  const float inv = pow2_neg(eps);
  float v[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
  uint4 q;
  q.x = cvt_e4m3x4(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv);
  q.y = cvt_e4m3x4(v[4] * inv, v[5] * inv, v[6] * inv, v[7] * inv);
  q.z = cvt_e4m3x4(v[8] * inv, v[9] * inv, v[10] * inv, v[11] * inv);
  q.w = cvt_e4m3x4(v[12] * inv, v[13] * inv, v[14] * inv, v[15] * inv);
  __stcs(reinterpret_cast<uint4*>(p.a_q + static_cast<size_t>(it.row) * p.d + it.col), q);
  if ((lane & 7) == 0) p.a_sf[sf_index(it.row, it.col >> 7, J)] = static_cast<uint8_t>(eps + 127);
}

__global__ void __launch_bounds__(kPermWarps * 32) permute_pad_kernel(const PermuteParams p) {
  const int lane = threadIdx.x & 31;
  const int chunks = (p.d + 511) >> 9;
  const int J = ((p.d >> 7) + 3) >> 2;
  pdl_trigger();
  pdl_wait();
  const int m_pad = min(*p.m_pad, p.M_cap);
  // Item g = row * chunks + chunk; this warp takes g0, g0 + S, g0 + 2S, ... (S warps in the grid),
  // two per trip.  Row and chunk of both are stepped by 2S with a carry instead of divided out.
  const long long S = static_cast<long long>(gridDim.x) * kPermWarps;
  const long long g0 = static_cast<long long>(blockIdx.x) * kPermWarps + (threadIdx.x >> 5);
  int row_a = static_cast<int>(g0 / chunks), ch_a = static_cast<int>(g0 % chunks);
  int row_b = static_cast<int>((g0 + S) / chunks), ch_b = static_cast<int>((g0 + S) % chunks);
  const int step_r = static_cast<int>((2 * S) / chunks), step_c = static_cast<int>((2 * S) % chunks);
  while (row_a < m_pad) {
    PermItem a, b;
    perm_load(p, row_a, ch_a, true, lane, a);
    perm_load(p, row_b, ch_b, row_b < m_pad, lane, b);
    perm_gather(p, a);
    perm_gather(p, b);
    perm_finish(p, a, lane, J);
    if (b.live) perm_finish(p, b, lane, J);
    row_a += step_r; ch_a += step_c;
    if (ch_a >= chunks) { ch_a -= chunks; ++row_a; }
    row_b += step_r; ch_b += step_c;
    if (ch_b >= chunks) { ch_b -= chunks; ++row_b; }
  }
}

// bf16 variant of step 2: the gathered rows stay bf16 (no quantiser); rows without a pair are zero.
// One warp per (row, 512-byte chunk), 16 bytes per lane.
__global__ void __launch_bounds__(kPermWarps * 32) permute_pad_bf16_kernel(const PermuteParams p, __nv_bfloat16* a) {
  const int lane = threadIdx.x & 31;
  const int row_bytes = 2 * p.d;
  const int chunks = (row_bytes + 511) >> 9;
  pdl_trigger();
  pdl_wait();
  const int m_pad = min(*p.m_pad, p.M_cap);
  const long long n_items = static_cast<long long>(m_pad) * chunks;
  const long long stride = static_cast<long long>(gridDim.x) * kPermWarps;
  for (long long gw = static_cast<long long>(blockIdx.x) * kPermWarps + (threadIdx.x >> 5); gw < n_items; gw += stride) {
    const int row = static_cast<int>(gw / chunks);
    const int off = static_cast<int>(gw % chunks) * 512 + lane * 16;
    if (off >= row_bytes) continue;
    const int pair = __ldg(p.row_pair + row);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (pair >= 0)
      v = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(p.x) +
                                                static_cast<size_t>(pair / p.k) * row_bytes + off));
    __stcs(reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(a) + static_cast<size_t>(row) * row_bytes + off), v);
  }
}

cudaError_t launch_permute_pad_bf16(const PermuteParams& p, __nv_bfloat16* a, int num_sms, cudaStream_t stream) {
  const long long warps = static_cast<long long>(p.M_cap) * ((2 * p.d + 511) >> 9);
  long long blocks = (warps + kPermWarps - 1) / kPermWarps;
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 8;
  if (blocks > cap) blocks = cap;
  return launch_pdl(permute_pad_bf16_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(kPermWarps * 32), 0, stream, p, a);
}

cudaError_t launch_permute_pad(const PermuteParams& p, int num_sms, cudaStream_t stream) {
  const long long warps = static_cast<long long>(p.M_cap) * ((p.d + 511) >> 9);
  long long blocks = (warps + kPermWarps - 1) / kPermWarps;
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 6;   // 6 CTAs of 8 warps are resident per SM at 40 registers
  if (blocks > cap) blocks = cap;
  return launch_pdl(permute_pad_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(kPermWarps * 32), 0, stream, p);
}

}  // namespace tempo
