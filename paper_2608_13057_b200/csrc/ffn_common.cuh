// Building blocks of the fused FFN kernel: tile geometry, PTX wrappers for mbarriers, bulk/tensor
// copies and the tcgen05 instructions, shared-memory and instruction descriptors, and the static
// tile assignment.
#pragma once

#include <cuda.h>

#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kBlockK = 128;
constexpr int kBlockN = 256;
constexpr int kABytes = kTileM * kBlockK;                 // 16 KB
constexpr int kBBytes = kBlockN * kBlockK;                // 32 KB
constexpr int kSfaBytes = 512;
constexpr int kSfbBytes = 1024;
constexpr int kTileOverhead = 5;                          // per-tile fixed cost in K-block steps (ramp + epilogue)
constexpr int kTmemCols = 512;
constexpr int kSfCol0 = 256;                              // scale slot s: A at 256+16s, B at 260+16s
constexpr int kMaxSlots = 1024;
constexpr int kStoreBytes = 32 * 128;                       // per-warp staging of a TMA store: 32 rows x 128 bytes


// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Ampere-style asynchronous copies (global -> shared, any destination address): 16 bytes past L1, or 4
// bytes; bytes beyond src_bytes are zero-filled (src_bytes = 0 reads nothing).
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait (limit in ns).  Returns false if the CTA is aborting (this wait or another one ran out of time).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
// Same copy with an L2 evict-first hint: for weight tiles that are read once per launch.
__device__ __forceinline__ void bulk_load_stream(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
// TMA tensor store of a 32-row x 128-byte box from (swizzled) shared memory, bulk-group completion.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_sf(uint32_t tmem_addr, uint64_t desc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem_addr), "l"(desc) : "memory");
}
__device__ __forceinline__ void tc_mma_mxf8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
      : "memory");
}
// bf16 x bf16 -> fp32, no scales (kind::f16 takes f16 or bf16 operands, chosen in the descriptor).
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Named barrier of two warps (64 threads).
__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }
// Compiler-level pin: the 32 values are treated as produced here, so nothing computed from them
// can be scheduled above this point.
__device__ __forceinline__ void pin32(uint32_t (&r)[32]) {
#pragma unroll
  for (int i = 0; i < 32; i += 8)
    asm volatile("" : "+r"(r[i]), "+r"(r[i + 1]), "+r"(r[i + 2]), "+r"(r[i + 3]), "+r"(r[i + 4]), "+r"(r[i + 5]),
                      "+r"(r[i + 6]), "+r"(r[i + 7])
                 :: "memory");
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 128 bytes, groups of
// 8 rows 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3fffu) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Descriptor of a 32-row x 16-byte scale atom (no swizzle, 8-row groups 128 bytes apart).
__device__ __forceinline__ uint64_t smem_desc_sf(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3fffu) | (static_cast<uint64_t>(128 >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::mxf8f6f4.block_scale: A, B e4m3 (format 0), both K-major,
// N >> 3 at bit 17, UE8M0 scales (bit 23), M >> 4 at bit 24; scale ids at bits 4 (B) and 29 (A).
__device__ __forceinline__ uint32_t instr_desc(int sf_id) {
  return (static_cast<uint32_t>(kBlockN >> 3) << 17) | (1u << 23) | (static_cast<uint32_t>(kTileM >> 4) << 24) |
         (static_cast<uint32_t>(sf_id) << 29) | (static_cast<uint32_t>(sf_id) << 4);
}

// Instruction descriptor of kind::f16 with bf16 operands: fp32 accumulator (1 at bit 4), A and B
// bf16 (1 at bits 7 and 10), both K-major, N >> 3 at bit 17, M >> 4 at bit 24.
__device__ __forceinline__ uint32_t instr_desc_bf16() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBlockN >> 3) << 17) |
         (static_cast<uint32_t>(kTileM >> 4) << 24);
}

struct WorkItem {
  int side;      // 0 gate/up, 1 down
  int inst, nt, row0, m_tiles;   // m_tiles: M-tiles of the instance (how often its B tiles are re-read)
};

// Tiles of one side are numbered instance-major, then N-tile, then M-tile, so CTAs running at the
// same time share B tiles through L2 and an instance's A rows stay L2-resident across its N-tiles.
//
// Two classes of instances are numbered separately: COLD ones (at most kColdTiles M-tiles: their
// weights are read from HBM and hardly re-used) and HOT ones (their weights are re-read from L2 by
// many M-tiles, so a tile is bound by the operand bytes an SM takes in).  A batch that has both
// (the hot/cold mix an EPLB-style placement leaves on a rank) would otherwise run its hot tiles
// with HBM idle and then its cold tiles with the tensor pipes idle.  TileOrder deals every wave of
// C tiles partly from the hot list and partly from the cold list, in the ratio at which a cold
// tile's weight stream and a hot tile's operand intake take the same time, so both run at once.
// With only one class present the order is the plain numbering.
constexpr int kColdTiles = 2;
constexpr int kColdShareNum = 80, kColdShareDen = 148;   // CTAs on cold tiles: HBM rate x hot-tile time / tile bytes

struct TileOrder {          // of one side
  int NT, n_hot, n_cold, C, Ch, Cc, W;
  __device__ TileOrder(int NT_, int hot_tiles, int cold_tiles, int C_) {
    NT = NT_; C = C_;
    n_hot = hot_tiles * NT; n_cold = cold_tiles * NT;
    Cc = (n_hot == 0 || n_cold == 0) ? 0 : max(1, min(C - 1, (C * kColdShareNum) / kColdShareDen));
    Ch = C - Cc;
    W = Cc == 0 ? 0 : min(n_hot / Ch, n_cold / Cc);      // waves dealt from both lists
  }
  // v-th tile of the side -> (class, index in the class's list)
  __device__ void map(int v, bool& cold, int& k) const {
    if (n_cold == 0) { cold = false; k = v; return; }
    if (n_hot == 0) { cold = true; k = v; return; }
    if (v < W * C) {
      const int w = v / C, j = v - w * C;
      if (j < Ch) { cold = false; k = w * Ch + j; } else { cold = true; k = w * Cc + (j - Ch); }
      return;
    }
    const int r = v - W * C, rem_hot = n_hot - W * Ch;     // what is left: hot first, then cold
    if (r < rem_hot) { cold = false; k = W * Ch + r; } else { cold = true; k = W * Cc + (r - rem_hot); }
  }
};

// M-tiles of the class before instance i: cold_before[i] counts the tiles of cold instances.
__device__ __forceinline__ int class_before(const int* toff, const uint16_t* cold_before, bool cold, int i) {
  return cold ? static_cast<int>(cold_before[i]) : toff[i] - static_cast<int>(cold_before[i]);
}

__device__ __forceinline__ WorkItem decode_item(int side, int v, const int* toff, const uint16_t* cold_before, int G,
                                                const TileOrder& order, int stride_tiles = 0) {
  bool cold;
  int k;
  order.map(v, cold, k);
  const int NT = order.NT;
  int lo = 0, hi = G - 1;
  while (lo < hi) {                       // first i with NT * class_before(i+1) > k
    const int mid = (lo + hi) >> 1;
    if (NT * class_before(toff, cold_before, cold, mid + 1) > k) hi = mid; else lo = mid + 1;
  }
  const int local = k - NT * class_before(toff, cold_before, cold, lo);
  const int Mi = toff[lo + 1] - toff[lo];
  WorkItem w;
  w.side = side;
  w.inst = lo;
  w.nt = local / Mi;
  w.row0 = ((stride_tiles > 0 ? lo * stride_tiles : toff[lo]) + local % Mi) * kTileM;   // masked layout: fixed stride
  w.m_tiles = Mi;
  return w;
}

// Static tile assignment, the same arithmetic in every role of every CTA.
//   gate/up tiles: x = c, c + C, ...  (n1 tiles; the first r1 = n1 % C CTAs get one more)
//   down tiles:    dealt in rounds.  The CTAs WITHOUT the extra gate/up tile ("light") take part
//                  in every round, the others only from round `lead` on, where `lead` is the extra
//                  tile's cost in down tiles - so every CTA streams about the same bytes.
struct TileIter {
  int c, C, n1, n2, r1, light, lead;
  int i1, round;
  __device__ TileIter(int c_, int C_, int n1_, int n2_, int Kb1, int Kb2) {
    c = c_; C = C_; n1 = n1_; n2 = n2_;
    r1 = n1 % C;
    light = C - r1;
    lead = (r1 == 0 || n2 == 0) ? 0 : (2 * (Kb1 + kTileOverhead) + (Kb2 + kTileOverhead)) / (2 * (Kb2 + kTileOverhead));
    i1 = c; round = 0;
  }
  // side and tile number of this CTA's next tile; false when it has none left
  __device__ bool next(int& side, int& x) {
    if (i1 < n1) { side = 0; x = i1; i1 += C; return true; }
    for (;;) {
      int y;
      if (round < lead) {
        if (c < r1) { round = lead; continue; }           // heavy CTAs skip the lead rounds
        y = round * light + (c - r1);
      } else {
        y = lead * light + (round - lead) * C + c;
      }
      ++round;
      if (y >= n2) return false;
      side = 1; x = y;
      return true;
    }
  }
};

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}


}  // namespace tempo
