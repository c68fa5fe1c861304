// One-time weight re-layout for the grouped GEMM kernels (off the hot path).
//
// Packed blob, in order (every section 1024-byte aligned):
//   W13t   u8 [G][f/128][d/128][256][128]   B tiles of the gate/up GEMM.  Tile (jb, kb) holds, for
//          the 128-column block jb of H, 128 gate rows then 128 up rows (so one tile feeds both
//          halves of SwiGLU) times the 128 K-bytes of block kb, stored exactly as the tensor core
//          reads them from shared memory: rows of 128 bytes, 16-byte chunk c of row r at chunk
//          position c ^ (r & 7) (the 128-byte swizzle).  A tile is one contiguous 32 KB read and
//          the tiles of one (instance, jb) follow each other along K: the weight stream of the
//          flat regime is sequential in HBM.
//   W2t    u8 [G][ceil(d/256)][f/128][256][128]   same for the down GEMM (rows beyond d are zero)
//   SF13   u8 [G][f/128][J1][2][512]   UE8M0 scale atoms of W13t tiles (gate atom, up atom)
//   SF2    u8 [G][ceil(d/256)][J2][2][512]   scale atoms of W2t tiles (two 128-row blocks per tile)
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
  L.off_sf13 = align1k(L.off_w2 + static_cast<size_t>(G) * L.NT2 * 256 * f);
  L.off_sf2 = align1k(L.off_sf13 + static_cast<size_t>(G) * L.NT1 * L.J1 * 1024);
  L.total = align1k(L.off_sf2 + static_cast<size_t>(G) * L.NT2 * L.J2 * 1024);
  return L;
}

// One thread per 16-byte chunk of the packed tiles.  mode 0: W13 [G][2f][d] -> W13t; mode 1: W2
// [G][d][f] -> W2t.  n_rows = source rows per instance, K = source row length.
__global__ void pack_tiles_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int G, int NT, int Kb,
                                  int n_rows, int K, int mode) {
  const size_t total = static_cast<size_t>(G) * NT * Kb * 256 * 8;
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(i & 7);
    const int r = static_cast<int>((i >> 3) & 255);
    size_t rest = i >> 11;
    const int kb = static_cast<int>(rest % Kb);
    rest /= Kb;
    const int nt = static_cast<int>(rest % NT);
    const int g = static_cast<int>(rest / NT);
    int srow;
    if (mode == 0) srow = (r < 128 ? 0 : n_rows / 2) + nt * 128 + (r & 127);
    else srow = nt * 256 + r;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (srow < n_rows)
      v = *reinterpret_cast<const uint4*>(src + (static_cast<size_t>(g) * n_rows + srow) * K + kb * 128 + c * 16);
    const size_t tile = (static_cast<size_t>(g) * NT + nt) * Kb + kb;
    *reinterpret_cast<uint4*>(dst + tile * 32768 + r * 128 + ((c ^ (r & 7)) << 4)) = v;
  }
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

// bf16 variant: W13 bf16 [G][2f][d] and W2 bf16 [G][d][f] into tiles of 256 rows x 64 values (128
// bytes per row, 32 KB per tile), same row interleave, swizzle and tile order as the fp8 blob:
//   W13t [G][f/128][d/64][256][128 B], then W2t [G][ceil(d/256)][f/64][256][128 B]; no scales.
PackLayout pack_layout_bf16(int G, int d, int f) {
  PackLayout L{};
  L.NT1 = f / 128;
  L.NT2 = (d + 255) / 256;
  L.off_w13 = 0;
  L.off_w2 = align1k(static_cast<size_t>(G) * 2 * f * d * 2);
  L.total = align1k(L.off_w2 + static_cast<size_t>(G) * L.NT2 * 256 * f * 2);
  L.off_sf13 = L.off_sf2 = L.total;
  return L;
}

// One thread per 16-byte chunk (8 values).  Kb = K / 64.
__global__ void pack_tiles_bf16_kernel(const __nv_bfloat16* __restrict__ src, uint8_t* __restrict__ dst, int G, int NT,
                                       int Kb, int n_rows, int K, int mode) {
  const size_t total = static_cast<size_t>(G) * NT * Kb * 256 * 8;
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(i & 7);
    const int r = static_cast<int>((i >> 3) & 255);
    size_t rest = i >> 11;
    const int kb = static_cast<int>(rest % Kb);
    rest /= Kb;
    const int nt = static_cast<int>(rest % NT);
    const int g = static_cast<int>(rest / NT);
    int srow;
    if (mode == 0) srow = (r < 128 ? 0 : n_rows / 2) + nt * 128 + (r & 127);
    else srow = nt * 256 + r;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (srow < n_rows)
      v = *reinterpret_cast<const uint4*>(src + (static_cast<size_t>(g) * n_rows + srow) * K + kb * 64 + c * 8);
    const size_t tile = (static_cast<size_t>(g) * NT + nt) * Kb + kb;
    *reinterpret_cast<uint4*>(dst + tile * 32768 + r * 128 + ((c ^ (r & 7)) << 4)) = v;
  }
}

cudaError_t launch_pack_bf16(int G, int d, int f, const __nv_bfloat16* w13, const __nv_bfloat16* w2, uint8_t* packed,
                             cudaStream_t stream) {
  const PackLayout L = pack_layout_bf16(G, d, f);
  pack_tiles_bf16_kernel<<<2368, 256, 0, stream>>>(w13, packed + L.off_w13, G, L.NT1, d / 64, 2 * f, d, 0);
  pack_tiles_bf16_kernel<<<2368, 256, 0, stream>>>(w2, packed + L.off_w2, G, L.NT2, f / 64, d, f, 1);
  return cudaGetLastError();
}

cudaError_t launch_pack(int G, int d, int f, const uint8_t* w13_q, const float* w13_s, const uint8_t* w2_q,
                        const float* w2_s, uint8_t* packed, uint32_t* status, cudaStream_t stream) {
  const PackLayout L = pack_layout(G, d, f);
  pack_tiles_kernel<<<2368, 256, 0, stream>>>(w13_q, packed + L.off_w13, G, L.NT1, d / 128, 2 * f, d, 0);
  pack_tiles_kernel<<<2368, 256, 0, stream>>>(w2_q, packed + L.off_w2, G, L.NT2, f / 128, d, f, 1);
  pack_sf_kernel<<<G * L.NT1 * L.J1 * 2, 128, 0, stream>>>(w13_s, packed + L.off_sf13, G, 2 * f / 128, d / 128,
                                                          L.NT1, L.J1, 0, status);
  pack_sf_kernel<<<G * L.NT2 * L.J2 * 2, 128, 0, stream>>>(w2_s, packed + L.off_sf2, G, d / 128, f / 128, L.NT2,
                                                          L.J2, 1, status);
  return cudaGetLastError();
}

}  // namespace tempo
