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

// Token of a pair: a shift when k is a power of two (kshift >= 0), a division otherwise.
__device__ __forceinline__ int pair_token(int pair, int k, int kshift) { return kshift >= 0 ? pair >> kshift : pair / k; }

__device__ __forceinline__ int shift_of(int k) { return (k & (k - 1)) == 0 ? __ffs(k) - 1 : -1; }

__device__ __forceinline__ void perm_gather(const PermuteParams& p, PermItem& it, int kshift) {
  if (it.in && it.pair >= 0) {
    const __nv_bfloat16* src = p.x + static_cast<size_t>(pair_token(it.pair, p.k, kshift)) * p.d + it.col;
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
  const int kshift = shift_of(p.k);
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
    perm_gather(p, a, kshift);
    perm_gather(p, b, kshift);
    perm_finish(p, a, lane, J);
    if (b.live) perm_finish(p, b, lane, J);
    row_a += step_r; ch_a += step_c;
    if (ch_a >= chunks) { ch_a -= chunks; ++row_a; }
    row_b += step_r; ch_b += step_c;
    if (ch_b >= chunks) { ch_b -= chunks; ++row_b; }
  }
}

// Token-major form.  Phase A: one warp per (token, 512-column chunk), two in flight: a lane loads its 32
// bytes of x and (lanes below k) one pair -> row entry, the block maxima and codes are computed ONCE and
// stored to the row of every local pair of the token - x is read from HBM once, and the row index and
// the activations arrive together instead of one after the other.  Phase B: rows of the padded
// layout that hold no pair are filled with zero codes and scale 1.
struct TokItem {
  int t, col, row;      // row: this lane's pair -> row entry (lanes >= k: -1)
  bool live, in;
  uint4 lo, hi;
};

__device__ __forceinline__ void tok_load(const PermuteParams& p, int t, int chunk, bool live, int lane, TokItem& it) {
  it.live = live;
  it.t = live ? t : 0;
  it.col = live ? chunk * 512 + lane * 16 : 0;
  it.in = live && it.col < p.d;
  it.row = (live && lane < p.k) ? __ldg(p.pair_row + static_cast<size_t>(it.t) * p.k + lane) : -1;
  it.lo = make_uint4(0, 0, 0, 0);
  it.hi = make_uint4(0, 0, 0, 0);
  if (it.in) {
    const __nv_bfloat16* src = p.x + static_cast<size_t>(it.t) * p.d + it.col;
    it.lo = __ldcs(reinterpret_cast<const uint4*>(src));
    it.hi = __ldcs(reinterpret_cast<const uint4*>(src + 8));
  }
}

__device__ __forceinline__ void tok_finish(const PermuteParams& p, const TokItem& it, int lane, int J, int m_pad) {
  if (__ballot_sync(0xffffffffu, it.row >= 0) == 0) return;     // no local pair: nothing to write
  const uint32_t w[8] = {it.lo.x, it.lo.y, it.lo.z, it.lo.w, it.hi.x, it.hi.y, it.hi.z, it.hi.w};
  __nv_bfloat162 m2 = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[0]));
#pragma unroll
  for (int i = 1; i < 8; ++i) m2 = __hmax2(m2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
  const uint32_t mbits = *reinterpret_cast<const uint32_t*>(&m2);
  float amax = fmaxf(__uint_as_float(mbits << 16), __uint_as_float(mbits & 0xffff0000u));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
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
  for (int s = 0; s < p.k; ++s) {
    const int row = __shfl_sync(0xffffffffu, it.row, s);
    if (row < 0 || row >= m_pad || !it.in) continue;            // row: warp-uniform
    __stcs(reinterpret_cast<uint4*>(p.a_q + static_cast<size_t>(row) * p.d + it.col), q);
    if ((lane & 7) == 0) p.a_sf[sf_index(row, it.col >> 7, J)] = static_cast<uint8_t>(eps + 127);
  }
}

__global__ void __launch_bounds__(kPermWarps * 32) permute_tokens_kernel(const PermuteParams p) {
  const int lane = threadIdx.x & 31;
  const int chunks = (p.d + 511) >> 9;
  const int J = ((p.d >> 7) + 3) >> 2;
  pdl_trigger();
  const long long S = static_cast<long long>(gridDim.x) * kPermWarps;
  const long long g0 = static_cast<long long>(blockIdx.x) * kPermWarps + (threadIdx.x >> 5);
  pdl_wait();
  // ---- phase A: tokens -----------------------------------------------------------------------
  {
    int t_a = static_cast<int>(g0 / chunks), ch_a = static_cast<int>(g0 % chunks);
    int t_b = static_cast<int>((g0 + S) / chunks), ch_b = static_cast<int>((g0 + S) % chunks);
    const int step_t = static_cast<int>((2 * S) / chunks), step_c = static_cast<int>((2 * S) % chunks);
    TokItem a, b;
    if (t_a < p.T) {
      tok_load(p, t_a, ch_a, true, lane, a);                    // issued together with the m_pad read below
      tok_load(p, t_b, ch_b, t_b < p.T, lane, b);
    }
    const int m_pad = min(*p.m_pad, p.M_cap);
    while (t_a < p.T) {
      tok_finish(p, a, lane, J, m_pad);
      if (b.live) tok_finish(p, b, lane, J, m_pad);
      t_a += step_t; ch_a += step_c;
      if (ch_a >= chunks) { ch_a -= chunks; ++t_a; }
      t_b += step_t; ch_b += step_c;
      if (ch_b >= chunks) { ch_b -= chunks; ++t_b; }
      if (t_a < p.T) {
        tok_load(p, t_a, ch_a, true, lane, a);
        tok_load(p, t_b, ch_b, t_b < p.T, lane, b);
      }
    }
  }
  // ---- phase B: rows without a pair ----------------------------------------------------------
  // One warp per (group of 32 rows, 512-column chunk), so the fill spreads over the whole grid.
  const int m_pad = min(*p.m_pad, p.M_cap);
  const long long groups = (m_pad + 31) >> 5;
  for (long long g = g0; g < groups * chunks; g += S) {
    const int base = static_cast<int>(g / chunks) * 32;
    const int col = static_cast<int>(g % chunks) * 512 + lane * 16;
    const int r = base + lane;
    bool pad = r < m_pad && __ldg(p.row_pair + r) < 0;
    if (pad && p.tile_inst != nullptr) pad = __ldg(p.tile_inst + (r >> 7)) >= 0;   // masked layout: used tiles only
    uint32_t todo = __ballot_sync(0xffffffffu, pad);
    if (col >= p.d) continue;
    while (todo) {
      const int row = base + __ffs(todo) - 1;
      todo &= todo - 1;
      __stcs(reinterpret_cast<uint4*>(p.a_q + static_cast<size_t>(row) * p.d + col), make_uint4(0, 0, 0, 0));
      if ((lane & 7) == 0) p.a_sf[sf_index(row, col >> 7, J)] = 127;
    }
  }
}

// One-wave form of the token-major walk, for batches small enough that every item gets a warp of its own
// (decode-sized): warps [0, T * chunks) take one (token, chunk) each, the warps after them one
// (group of kFillRows rows, chunk) of the zero fill, so nothing queues behind anything else and the kernel
// lasts one index + activation latency instead of the two or three round trips of a grid-stride walk
// (config 2: 5.5 -> 2.7 us from the end of the dispatch).  The next kernel is released after the wait: let in
// earlier, its CTAs sit resident through the previous step's tail, which cost more than their prologue saves.
constexpr int kFillRows = 16;

__global__ void __launch_bounds__(kPermWarps * 32) permute_wave_kernel(const PermuteParams p) {
  const int lane = threadIdx.x & 31;
  const int chunks = (p.d + 511) >> 9;
  const int J = ((p.d >> 7) + 3) >> 2;
  const long long S = static_cast<long long>(gridDim.x) * kPermWarps;
  const long long n_tok = static_cast<long long>(p.T) * chunks;
  const long long n_all = n_tok + static_cast<long long>((p.M_cap + kFillRows - 1) / kFillRows) * chunks;
  pdl_wait();
  pdl_trigger();
  // (the grid holds a warp per item up to 4 CTAs per SM; beyond that a warp takes two or three items in turn)
  for (long long w = static_cast<long long>(blockIdx.x) * kPermWarps + (threadIdx.x >> 5); w < n_all; w += S) {
    if (w < n_tok) {
      TokItem a;
      tok_load(p, static_cast<int>(w / chunks), static_cast<int>(w % chunks), true, lane, a);
      const int m_pad = min(*p.m_pad, p.M_cap);
      tok_finish(p, a, lane, J, m_pad);
      continue;
    }
    const long long g = w - n_tok;
    const int base = static_cast<int>(g / chunks) * kFillRows;
    const int col = static_cast<int>(g % chunks) * 512 + lane * 16;
    const int r = base + lane;
    const bool mine = lane < kFillRows && r < p.M_cap;
    const int pair = mine ? __ldg(p.row_pair + r) : 0;
    // masked layout: used tiles only (tile_inst has M_cap / 128 entries)
    const int inst = (mine && p.tile_inst != nullptr && (r >> 7) < p.M_cap / kTileM) ? __ldg(p.tile_inst + (r >> 7)) : 0;
    const int m_pad = min(*p.m_pad, p.M_cap);
    uint32_t todo = __ballot_sync(0xffffffffu, mine && r < m_pad && pair < 0 && inst >= 0);
    if (col >= p.d) continue;
    while (todo) {
      const int row = base + __ffs(todo) - 1;
      todo &= todo - 1;
      __stcs(reinterpret_cast<uint4*>(p.a_q + static_cast<size_t>(row) * p.d + col), make_uint4(0, 0, 0, 0));
      if ((lane & 7) == 0) p.a_sf[sf_index(row, col >> 7, J)] = 127;
    }
  }
}

// Step 2 without the layout: quantise every live token row ONCE, in token order (x_q[t,:], one scale byte per
// 128 columns in x_sf[t, :]), for the FFN entry point that gathers its rows itself (tempo_grouped_ffn_gather).
// Nothing here depends on step 1, so the kernel does not wait for it at its start: launched behind the
// dispatch kernel it runs beside it on the SMs the dispatch cluster leaves free.  It waits for its predecessor
// only at its end, so that "this kernel is complete" still implies "step 1 is complete" for the kernel after it.
// One warp per (token, 512-column chunk), four in flight, grid-stride.
constexpr int kQuantInFlight = 4;

__global__ void __launch_bounds__(kPermWarps * 32) quantize_tokens_kernel(const QuantizeParams p) {
  const int lane = threadIdx.x & 31;
  const int chunks = (p.d + 511) >> 9;
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));     // an input of the step, not a result of step 1
  const long long S = static_cast<long long>(gridDim.x) * kPermWarps;
  const long long g0 = static_cast<long long>(blockIdx.x) * kPermWarps + (threadIdx.x >> 5);
  const long long n_items = static_cast<long long>(nv) * chunks;
  for (long long g = g0; g < n_items; g += kQuantInFlight * S) {
    uint4 lo[kQuantInFlight], hi[kQuantInFlight];
    int t[kQuantInFlight], col[kQuantInFlight];
    bool in[kQuantInFlight];
#pragma unroll
    for (int u = 0; u < kQuantInFlight; ++u) {
      const long long gi = g + u * S;
      const bool live = gi < n_items;
      t[u] = live ? static_cast<int>(gi / chunks) : 0;
      col[u] = live ? static_cast<int>(gi % chunks) * 512 + lane * 16 : 0;
      in[u] = live && col[u] < p.d;
      lo[u] = make_uint4(0, 0, 0, 0);
      hi[u] = make_uint4(0, 0, 0, 0);
      if (in[u]) {
        const __nv_bfloat16* src = p.x + static_cast<size_t>(t[u]) * p.d + col[u];
        lo[u] = __ldcs(reinterpret_cast<const uint4*>(src));
        hi[u] = __ldcs(reinterpret_cast<const uint4*>(src + 8));
      }
    }
#pragma unroll
    for (int u = 0; u < kQuantInFlight; ++u) {
      const uint32_t w[8] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w, hi[u].x, hi[u].y, hi[u].z, hi[u].w};
      __nv_bfloat162 m2 = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[0]));
#pragma unroll
      for (int i = 1; i < 8; ++i) m2 = __hmax2(m2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
      const uint32_t mbits = *reinterpret_cast<const uint32_t*>(&m2);
      float amax = fmaxf(__uint_as_float(mbits << 16), __uint_as_float(mbits & 0xffff0000u));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
      if (!in[u]) continue;
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
      *reinterpret_cast<uint4*>(p.x_q + static_cast<size_t>(t[u]) * p.d + col[u]) = q;     // re-read soon: keep it in L2
      if ((lane & 7) == 0) p.x_sf[static_cast<size_t>(t[u]) * p.sf_stride + (col[u] >> 7)] = static_cast<uint8_t>(eps + 127);
    }
  }
  pdl_wait();
  pdl_trigger();
}

cudaError_t launch_quantize_tokens(const QuantizeParams& p, int num_sms, cudaStream_t stream) {
  const long long warps = static_cast<long long>(p.T) * ((p.d + 511) >> 9);
  long long blocks = (warps + kQuantInFlight * kPermWarps - 1) / (kQuantInFlight * kPermWarps);
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 6;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return launch_pdl(quantize_tokens_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(kPermWarps * 32), 0, stream, p);
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

static cudaError_t launch_permute_tokens(const PermuteParams& p, int num_sms, cudaStream_t stream) {
  const long long chunks = (p.d + 511) >> 9;
  const long long warps = max(static_cast<long long>(p.T) * chunks, (static_cast<long long>(p.M_cap) / 32 + 1) * chunks);
  long long blocks = (warps + 2 * kPermWarps - 1) / (2 * kPermWarps);        // two items per warp per trip
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 6;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return launch_pdl(permute_tokens_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(kPermWarps * 32), 0, stream, p);
}

cudaError_t launch_permute_pad(const PermuteParams& p, int num_sms, cudaStream_t stream) {
  // Token-major pays when the rows of x no longer stay in L2 between the (up to k) gathers of a token:
  // measured on B200, config 4 (x = 117 MB) 150 -> 100 us; with x = 34 MB (config 3) the gathers hit L2
  // anyway and the row-major walk is 2 us faster.
  constexpr size_t kTokenMajorBytes = 48u << 20;
  if (p.pair_row != nullptr) {
    // a warp per item, all of them resident at once (4 CTAs per SM leave room beside the dispatch cluster);
    // larger batches keep that grid and give a warp several items
    const long long chunks = (p.d + 511) >> 9;
    const long long warps = (static_cast<long long>(p.T) + (p.M_cap + kFillRows - 1) / kFillRows) * chunks;
    const long long blocks = max(1LL, (warps + kPermWarps - 1) / kPermWarps);
    const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 4;
    // up to six items per warp it still beats the row walk (measured: T = 1024 -1.2 us, T = 2048 -3 us per block;
    // at T = 4096, ten items per warp, it is 1.4 us behind)
    if (blocks <= 6 * cap)
      return launch_pdl(permute_wave_kernel, dim3(static_cast<unsigned int>(min(blocks, cap))), dim3(kPermWarps * 32), 0,
                        stream, p);
  }
  if (p.pair_row != nullptr && (p.tile_inst != nullptr || static_cast<size_t>(p.T) * p.d * 2 > kTokenMajorBytes))
    return launch_permute_tokens(p, num_sms, stream);                 // the masked layout always walks the tokens
  const long long warps = static_cast<long long>(p.M_cap) * ((p.d + 511) >> 9);
  long long blocks = (warps + kPermWarps - 1) / kPermWarps;
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 6;   // 6 CTAs of 8 warps are resident per SM at 40 registers
  if (blocks > cap) blocks = cap;
  return launch_pdl(permute_pad_kernel, dim3(static_cast<unsigned int>(blocks)), dim3(kPermWarps * 32), 0, stream, p);
}

}  // namespace tempo
