// One-time weight re-layout for the grouped GEMM kernels (off the hot path).
//
// Packed blob, in order (every section 1024-byte aligned):
//   W13p   u8 [G][f/128][256][d]   per 128-column block jb of H: 128 gate rows then 128 up rows,
//                                  so one 256-row B tile feeds both halves of SwiGLU
//   W2p    u8 [G][d][f]            unchanged order
//   SF13   u8 [G][f/128][J1][2][512]   UE8M0 scale atoms of W13p tiles (gate atom, up atom)
//   SF2    u8 [G][ceil(d/256)][J2][2][512]   scale atoms of W2 tiles (two 128-row blocks per tile)
// An atom covers 128 rows x 4 K-blocks in the order the tensor core's scale copy consumes:
// word (row%32)*4 + row/32 holds the 4 scale bytes of that row.  Weight scales are per 128x128
// block, so all 128 rows of an atom carry the same word.  J = ceil((K/128)/4).
#include "tempo_kernels.cuh"

namespace tempo {


__host__ __device__ inline size_t align1k(size_t v) { return (v + 1023) & ~static_cast<size_t>(1023); }

PackLayout pack_layout(int G, int d, int f) {
  PackLayout L;
  L.J1 = ((d / 128) + 3) / 4;
  L.J2 = ((f / 128) + 3) / 4;
  L.NT1 = f / 128;
  L.NT2 = (d + 255) / 256;
  L.off_w13 = 0;
  L.off_w2 = align1k(L.off_w13 + static_cast<size_t>(G) * 2 * f * d);
  L.off_sf13 = align1k(L.off_w2 + static_cast<size_t>(G) * d * f);
  L.off_sf2 = align1k(L.off_sf13 + static_cast<size_t>(G) * L.NT1 * L.J1 * 1024);
  L.total = align1k(L.off_sf2 + static_cast<size_t>(G) * L.NT2 * L.J2 * 1024);
  return L;
}

// rows of W13 are permuted: packed row (g, jb, half, r) <- source row (g, half*f + jb*128 + r)
__global__ void pack_w13_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int G, int d, int f) {
  const size_t chunks_per_row = d / 16;
  const size_t total = static_cast<size_t>(G) * 2 * f * chunks_per_row;
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t prow = i / chunks_per_row, c = i % chunks_per_row;
    const int g = static_cast<int>(prow / (2 * f));
    const int within = static_cast<int>(prow % (2 * f));
    const int jb = within / 256, half = (within % 256) / 128, r = within % 128;
    const size_t srow = static_cast<size_t>(g) * 2 * f + static_cast<size_t>(half) * f + jb * 128 + r;
    reinterpret_cast<uint4*>(dst)[prow * chunks_per_row + c] = reinterpret_cast<const uint4*>(src)[srow * chunks_per_row + c];
  }
}

__global__ void copy16_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<size_t>(gridDim.x) * blockDim.x)
    dst[i] = src[i];
}

__device__ __forceinline__ uint32_t ue8m0_of(float s, uint32_t* bad) {
  const uint32_t bits = __float_as_uint(s);
  const uint32_t ef = (bits >> 23) & 0xffu;
  if ((bits & 0x807fffffu) != 0 || ef == 0 || ef == 255) *bad = 1;
  return ef;
}

// scales: f32 [G][n_blocks][k_blocks].  One thread per (g, tile, j, atom): builds the word and
// writes it 128 times.  mode 0: W13 (atom 0 = gate block jb, atom 1 = up block f/128 + jb);
// mode 1: W2 (atom a = 128-row block 2*tile + a, absent blocks get scale 1).
__global__ void pack_sf_kernel(const float* __restrict__ scales, uint8_t* __restrict__ dst, int G, int n_blocks,
                               int k_blocks, int tiles, int J, int mode, uint32_t* status) {
  const int total = G * tiles * J * 2;
  const int item = blockIdx.x;
  if (item >= total) return;
  const int atom = item & 1;
  const int j = (item >> 1) % J;
  const int tile = ((item >> 1) / J) % tiles;
  const int g = (item >> 1) / J / tiles;
  const int nb = mode == 0 ? (atom == 0 ? tile : n_blocks / 2 + tile) : 2 * tile + atom;
  uint32_t bad = 0, word = 0;
  for (int q = 0; q < 4; ++q) {
    const int kb = 4 * j + q;
    uint32_t b = 127;
    if (nb < n_blocks && kb < k_blocks)
      b = ue8m0_of(scales[(static_cast<size_t>(g) * n_blocks + nb) * k_blocks + kb], &bad);
    word |= b << (8 * q);
  }
  reinterpret_cast<uint32_t*>(dst)[static_cast<size_t>(item) * 128 + threadIdx.x] = word;
  if (bad && threadIdx.x == 0) atomicOr(status, static_cast<uint32_t>(TEMPO_STATUS_BAD_SCALE));
}

cudaError_t launch_pack(int G, int d, int f, const uint8_t* w13_q, const float* w13_s, const uint8_t* w2_q,
                        const float* w2_s, uint8_t* packed, uint32_t* status, cudaStream_t stream) {
  const PackLayout L = pack_layout(G, d, f);
  pack_w13_kernel<<<1184, 256, 0, stream>>>(w13_q, packed + L.off_w13, G, d, f);
  copy16_kernel<<<1184, 256, 0, stream>>>(reinterpret_cast<const uint4*>(w2_q),
                                          reinterpret_cast<uint4*>(packed + L.off_w2),
                                          static_cast<size_t>(G) * d * f / 16);
  pack_sf_kernel<<<G * L.NT1 * L.J1 * 2, 128, 0, stream>>>(w13_s, packed + L.off_sf13, G, 2 * f / 128, d / 128,
                                                          L.NT1, L.J1, 0, status);
  pack_sf_kernel<<<G * L.NT2 * L.J2 * 2, 128, 0, stream>>>(w2_s, packed + L.off_sf2, G, d / 128, f / 128, L.NT2,
                                                          L.J2, 1, status);
  return cudaGetLastError();
}

}  // namespace tempo
