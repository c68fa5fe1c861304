// Step 3: fp8 grouped SwiGLU FFN on the 5th-generation tensor cores (sm_100a), ONE persistent kernel.
//
// Two kinds of 128x256 output tiles:
//   gate/up  GU = A * W13t^T (128 gate + 128 up columns of one 128-column block of H), epilogue
//            H = silu(gate) * up, re-quantised to e4m3 with a 1x128 power-of-two scale;
//   down     Y = Hq * W2t^T, epilogue converts to bf16.
// This is the load-dependent term of the paper's cost model (Section 2.1, Eq. 1): with few rows
// per instance the kernel streams every activated instance's weights once (the floor b per
// instance), with many rows it is bound by the tensor pipe (beta per row, in 128-row tiles, Eq. 3).
// Both kinds run in the same launch so the weight stream has one ramp and one tail and the CTAs
// that run out of gate/up tiles go straight on to down tiles.  A down tile needs every H block
// of its 128 rows: the epilogue warps of a finished gate/up tile bump a per-M-tile counter, and
// only the ACTIVATION loads of a down tile wait for it (bounded); its weight loads never wait,
// so HBM keeps streaming.  The counters clean themselves: the last down tile of an M-tile to see
// the counter complete puts it back to zero.
//
// Per CTA (one per SM, 384 threads):
//   warp 0     weight producer: per K-block one contiguous 32 KB bulk copy of a pre-swizzled
//              packed B tile (+ two 512-byte scale atoms every 4th K-block) into a 4-stage ring
//   warp 2     activation producer: per K-block a 128x128 A tile (TMA tensor copy, 128-byte
//              swizzle) (+ one scale atom every 4th K-block); waits for H where needed
//   warp 3     dependency scout: runs ahead of warp 2 through the down tiles, watches the H counters
//   warp 1     MMA issuer: tcgen05.cp moves scale atoms into tensor memory, then four
//              tcgen05.mma.kind::mxf8f6f4.block_scale (M128 N256 K32) per K-block accumulate in
//              tensor memory; tcgen05.commit releases the stage / publishes the accumulator
//   warps 4-11 epilogue, two warps per tensor-memory lane quadrant, each taking half of a row's
//              columns: tcgen05.ld the raw accumulator into registers and hand tensor memory back
//              to the MMA issuer at once, then the math (the pair shares the row maximum through
//              shared memory), swizzled staging in shared memory, TMA tensor stores
// Scales are UE8M0 per 128 K-elements; the MMA takes one scale byte per row (A) and per column
// (B) for each K=32 step, so the four steps of a K-block select the same byte (scale id kb % 4).
//
// Every wait is bounded: after kWaitLimitNs the CTA raises an abort flag, all roles leave their
// loops, TEMPO_STATUS_TIMEOUT is set and tensor memory is freed.
#include <cuda.h>

#include "tempo_kernels.cuh"

namespace tempo {

constexpr int kStages = 4;
constexpr int kBlockK = 128;
constexpr int kBlockN = 256;
constexpr int kABytes = kTileM * kBlockK;                 // 16 KB
constexpr int kBBytes = kBlockN * kBlockK;                // 32 KB
constexpr int kSfaBytes = 512;
constexpr int kSfbBytes = 1024;
constexpr int kStageBytes = kABytes + kBBytes + 2048;     // 51200, a multiple of 1024
constexpr int kGemmThreads = 384;
constexpr int kEpiWarp0 = 4;                               // first of the 8 epilogue warps
constexpr int kTileOverhead = 5;                          // per-tile fixed cost in K-block steps (ramp + epilogue)
constexpr int kTmemCols = 512;
constexpr int kSfCol0 = 256;                              // scale slot s: A at 256+16s, B at 260+16s
constexpr int kMaxSlots = 1024;
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;
constexpr int kStoreBytes = 32 * 128;                       // per-warp staging of a TMA store: 32 rows x 128 bytes
constexpr size_t kGemmSmemBytes = static_cast<size_t>(kStages) * kStageBytes + 4 * kStoreBytes + 1024;


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
// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out of time).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
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

struct WorkItem {
  int side;      // 0 gate/up, 1 down
  int inst, nt, row0, m_tiles;   // m_tiles: M-tiles of the instance (how often its B tiles are re-read)
};

// Tiles of one side are numbered instance-major, then N-tile, then M-tile, so CTAs running at the
// same time share B tiles through L2 and an instance's A rows stay L2-resident across its N-tiles.
__device__ __forceinline__ WorkItem decode_item(int side, int x, const int* toff, int G, int NT) {
  int lo = 0, hi = G - 1;
  while (lo < hi) {                       // first i with NT * toff[i+1] > x
    const int mid = (lo + hi) >> 1;
    if (NT * toff[mid + 1] > x) hi = mid; else lo = mid + 1;
  }
  const int local = x - NT * toff[lo];
  const int Mi = toff[lo + 1] - toff[lo];
  WorkItem w;
  w.side = side;
  w.inst = lo;
  w.nt = local / Mi;
  w.row0 = (toff[lo] + local % Mi) * kTileM;
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

__global__ void __launch_bounds__(kGemmThreads, 1)
ffn_kernel(const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmA2,
           const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmY, const FfnParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t s_full[kStages];
  __shared__ __align__(8) uint64_t s_empty[kStages];
  __shared__ __align__(8) uint64_t s_acc_full;
  __shared__ __align__(8) uint64_t s_acc_empty;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort_storage;
  __shared__ int s_dep_storage;
  __shared__ int s_toff[kMaxSlots + 1];
  __shared__ float s_amax[2][2][kTileM];   // [tile parity][column half][row]: row maxima of the two half-row warps
  __shared__ int s_ok[2][4][2];             // [tile parity][quadrant][column half]: that warp's wait succeeded
  volatile int* s_abort = &s_abort_storage;
  volatile int* s_dep = &s_dep_storage;   // down tiles of this CTA whose H rows are known complete

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int G = p.G_max;
  pdl_trigger();
  // prologue that needs nothing from the previous kernel: barriers, tensor memory, descriptor fetch
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&s_full[s]), 2); mbar_init(smem_u32(&s_empty[s]), 1); }
    mbar_init(smem_u32(&s_acc_full), 1);
    mbar_init(smem_u32(&s_acc_empty), 8);
    s_abort_storage = 0;
    s_dep_storage = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA1)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA2)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmH)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();
  const int m_pad = max(0, min(*p.m_pad, p.M_cap)) & ~(kTileM - 1);
  const int m_tiles = m_pad / kTileM;
  const int n1 = (p.run_mask & 1) ? m_tiles * p.side[0].NT : 0;
  const int n2 = (p.run_mask & 2) ? m_tiles * p.side[1].NT : 0;
  const bool fused = p.run_mask == 3;
  const int Kb1 = p.side[0].Kb, Kb2 = p.side[1].Kb;

  for (int i = tid; i <= G; i += kGemmThreads) s_toff[i] = max(0, min(p.inst_off[i], m_pad)) >> 7;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;

  if (warp == 0) {
    // ------------------------------- weight producer ------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const GemmSide& gs = p.side[side];
        const WorkItem w = decode_item(side, x, s_toff, G, gs.NT);
        const uint8_t* sfb_src = gs.sfb + (static_cast<size_t>(w.inst) * gs.NT + w.nt) * gs.JK * kSfbBytes;
        const uint8_t* b_src = gs.wt + (static_cast<size_t>(w.inst) * gs.NT + w.nt) * gs.Kb * kBBytes;
        const bool stream_b = w.m_tiles <= 2;
        for (int kb = 0; kb < gs.Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort)) { ok = false; break; }
          const uint32_t full = smem_u32(&s_full[stage]);
          const uint32_t sB = smem_base + stage * kStageBytes + kABytes, sSF = sB + kBBytes;
          const bool with_sf = (kb & 3) == 0;
          mbar_arrive_expect_tx(full, kBBytes + (with_sf ? kSfbBytes : 0));
          if (stream_b) bulk_load_stream(sB, b_src + static_cast<size_t>(kb) * kBBytes, kBBytes, full);
          else bulk_load(sB, b_src + static_cast<size_t>(kb) * kBBytes, kBBytes, full);
          if (with_sf) bulk_load(sSF + kSfaBytes, sfb_src + static_cast<size_t>(kb >> 2) * kSfbBytes, kSfbBytes, full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------- activation producer --------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      int n_down = 0;
      bool ok = true;
      TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const GemmSide& gs = p.side[side];
        const WorkItem w = decode_item(side, x, s_toff, G, gs.NT);
        const uint8_t* sfa_src = gs.sfa + static_cast<size_t>(w.row0 >> 7) * gs.JK * kSfaBytes;
        const CUtensorMap* tm = side == 0 ? &tmA1 : &tmA2;
        if (side == 1 && fused) {
          // wait until the scout (warp 3) has seen every H block of these 128 rows complete
          ++n_down;
          unsigned long long t0 = 0;
          for (uint32_t spin = 0; *s_dep < n_down; ++spin) {
            if ((spin & 255u) == 255u) {
              if (*s_abort) { ok = false; break; }
              const unsigned long long now = global_timer_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > kWaitLimitNs) { *s_abort = 1; ok = false; break; }
            }
          }
          if (!ok) break;
          __threadfence();
          asm volatile("fence.proxy.async;" ::: "memory");   // H was written by ordinary stores, TMA reads it
        }
        for (int kb = 0; kb < gs.Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort)) { ok = false; break; }
          const uint32_t full = smem_u32(&s_full[stage]);
          const uint32_t sA = smem_base + stage * kStageBytes, sSF = sA + kABytes + kBBytes;
          const bool with_sf = (kb & 3) == 0;
          mbar_arrive_expect_tx(full, kABytes + (with_sf ? kSfaBytes : 0));
          tma_load_2d(sA, tm, full, kb * kBlockK, w.row0);
          if (with_sf) bulk_load(sSF, sfa_src + static_cast<size_t>(kb >> 2) * kSfaBytes, kSfaBytes, full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------- dependency scout -----------------------------------------
    // Runs ahead through this CTA's down tiles: waits (bounded) until the four epilogue warps of
    // every gate/up tile of the tile's 128 rows have published their H rows, then tells the
    // activation producer through s_dep.  The last down tile of an M-tile to get here puts the
    // two global counters back to zero, so the workspace is clean when the kernel ends.
    if (lane == 0 && fused) {
      TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
      int side, x, cleared = 0;
      const int want = 4 * p.side[0].NT;
      bool ok = true;
      while (ok && it.next(side, x)) {
        if (side == 0) continue;
        const WorkItem w = decode_item(1, x, s_toff, G, p.side[1].NT);
        const int tau = w.row0 >> 7;
        unsigned long long t0 = 0;
        for (uint32_t spin = 0; ld_acquire(p.ready + tau) < want; ++spin) {
          if ((spin & 63u) == 63u) {
            if (*s_abort) { ok = false; break; }
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) { *s_abort = 1; ok = false; break; }
          }
        }
        if (!ok) break;
        if (atomicAdd(p.done + tau, 1) == p.side[1].NT - 1) {
          atomicExch(p.ready + tau, 0);
          atomicExch(p.done + tau, 0);
        }
        __threadfence();
        *s_dep = ++cleared;
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -----------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, acc_phase = 0;
      bool ok = true;
      TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const int Kb = p.side[side].Kb;
        if (!mbar_wait(smem_u32(&s_acc_empty), acc_phase ^ 1u, s_abort)) break;
        tc_fence_after();
        for (int kb = 0; kb < Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_full[stage]), phase, s_abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sA = smem_base + stage * kStageBytes, sB = sA + kABytes, sSF = sB + kBBytes;
          const uint32_t sfa_t = tmem_base + kSfCol0 + 16u * ((kb >> 2) & 1);
          const uint32_t sfb_t = sfa_t + 4;
          if ((kb & 3) == 0) {
            tc_cp_sf(sfa_t, smem_desc_sf(sSF));
            tc_cp_sf(sfb_t, smem_desc_sf(sSF + kSfaBytes));
            tc_cp_sf(sfb_t + 4, smem_desc_sf(sSF + kSfaBytes + 512));
          }
          const uint32_t idesc = instr_desc(kb & 3);
          const uint64_t da = smem_desc_sw128(sA), db = smem_desc_sw128(sB);
#pragma unroll
          for (int ks = 0; ks < kBlockK / 32; ++ks)
            tc_mma_mxf8(tmem_base, da + 2u * ks, db + 2u * ks, idesc, sfa_t, sfb_t, (kb | ks) != 0 ? 1u : 0u);
          tc_commit(smem_u32(&s_empty[stage]));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(smem_u32(&s_acc_full));
        acc_phase ^= 1u;
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ------------------------------- epilogue --------------------------------------------------
    // Warps w and w + 4 read the same tensor-memory lane quadrant (rows quad*32 .. +31 of the tile)
    // and split each row's columns.  The accumulator is copied raw into registers and released
    // before any arithmetic, so the MMA issuer starts the next tile while this one is finished.
    // Results leave through a per-quadrant 4 KB staging buffer (32 rows x 128 bytes, 128-byte
    // swizzle so the 16-byte writes of a warp hit distinct banks; each warp of the pair fills its
    // 64-byte half of every row) and one TMA tensor store per buffer: the global writes are full
    // lines and do not compete with the producers' loads for the SM's load/store path.
    const int quad = warp & 3;                       // tensor-memory lanes this warp may read
    const int half = (warp - kEpiWarp0) >> 2;        // which half of the columns
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const uint32_t stage_buf = smem_base + kStages * kStageBytes + quad * kStoreBytes;
    const uint32_t my_line = stage_buf + lane * 128;
    const bool issuer = half == 0 && lane == 0;      // the one thread of the pair that owns the TMA stores
    const int pair_bar = 1 + quad;                   // named barrier of the pair (64 threads)
    const int r_in_tile = quad * 32 + lane;
    uint32_t acc_phase = 0;
    int par = 0;
    TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
    int side, x;
    while (it.next(side, x)) {
      const WorkItem w = decode_item(side, x, s_toff, G, p.side[side].NT);
      const int row = w.row0 + r_in_tile;
      // Both warps of a pair must take the same way out: they vote on the outcome of the wait.
      const bool ok = mbar_wait(smem_u32(&s_acc_full), acc_phase, s_abort);
      acc_phase ^= 1u;
      if (lane == 0) s_ok[par][quad][half] = ok ? 1 : 0;
      pair_sync(pair_bar);
      if (!(s_ok[par][quad][0] && s_ok[par][quad][1])) break;
      tc_fence_after();
      if (side == 0) {
        // gate columns [64*half, +64) and the matching up columns of this thread's row
        uint32_t g[2][32], u[2][32];
        tmem_ld32(taddr + half * 64, g[0]);
        tmem_ld32(taddr + half * 64 + 32, g[1]);
        tmem_ld32(taddr + 128 + half * 64, u[0]);
        tmem_ld32(taddr + 128 + half * 64 + 32, u[1]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_acc_empty));   // accumulator drained: the next tile may start
        pin32(g[0]); pin32(g[1]); pin32(u[0]); pin32(u[1]);   // keep the arithmetic below the release
        float h[64];
        float amax = 0.f;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float gv = __uint_as_float(g[c][i]), uv = __uint_as_float(u[c][i]);
            const float hv = __fdividef(gv, 1.f + __expf(-gv)) * uv;
            h[c * 32 + i] = hv;
            amax = fmaxf(amax, fabsf(hv));
          }
        }
        s_amax[par][half][r_in_tile] = amax;
        if (issuer) bulk_wait_read();                         // the previous store has left the buffer
        pair_sync(pair_bar);
        amax = fmaxf(amax, s_amax[par][half ^ 1][r_in_tile]);
        const int eps = pow2_scale_exponent(amax);
        const float inv = pow2_neg(eps);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 q;
          q.x = cvt_e4m3x4(h[16 * v + 0] * inv, h[16 * v + 1] * inv, h[16 * v + 2] * inv, h[16 * v + 3] * inv);
          q.y = cvt_e4m3x4(h[16 * v + 4] * inv, h[16 * v + 5] * inv, h[16 * v + 6] * inv, h[16 * v + 7] * inv);
          q.z = cvt_e4m3x4(h[16 * v + 8] * inv, h[16 * v + 9] * inv, h[16 * v + 10] * inv, h[16 * v + 11] * inv);
          q.w = cvt_e4m3x4(h[16 * v + 12] * inv, h[16 * v + 13] * inv, h[16 * v + 14] * inv, h[16 * v + 15] * inv);
          st_shared_v4(my_line + (((half * 4 + v) ^ (lane & 7)) << 4), q);
        }
        if (half == 0) p.h_sf[sf_index(row, w.nt, p.J_h)] = static_cast<uint8_t>(eps + 127);
        fence_async_smem();
        if (fused) __threadfence();                            // the scale byte, before the counter below
        pair_sync(pair_bar);
        if (issuer) {
          tma_store_2d(&tmH, stage_buf, w.nt * 128, w.row0 + quad * 32);
          bulk_commit();
          if (fused) {                                         // publish these 32 rows of the H block
            bulk_wait_all();
            asm volatile("fence.proxy.async;" ::: "memory");
            __threadfence();
            atomicAdd(p.ready + (w.row0 >> 7), 1);
          }
        }
      } else {
        // Of every 64-column group of the tile this thread takes 32 columns: [64*s + 32*half, +32).
        uint32_t a[4][32];
#pragma unroll
        for (int s = 0; s < 4; ++s) tmem_ld32(taddr + s * 64 + half * 32, a[s]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_acc_empty));
        pin32(a[0]); pin32(a[1]); pin32(a[2]); pin32(a[3]);
#pragma unroll
        for (int s = 0; s < 4; ++s) {                           // 64 columns = 128 bytes per row per store
          if (w.nt * kBlockN + s * 64 < p.d) {                  // same for the pair; the store clips at column d
            uint32_t packed[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 b =
                  __floats2bfloat162_rn(__uint_as_float(a[s][2 * i]), __uint_as_float(a[s][2 * i + 1]));
              packed[i] = *reinterpret_cast<const uint32_t*>(&b);
            }
            if (issuer) bulk_wait_read();
            pair_sync(pair_bar);
#pragma unroll
            for (int v = 0; v < 4; ++v)
              st_shared_v4(my_line + (((half * 4 + v) ^ (lane & 7)) << 4),
                           make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]));
            fence_async_smem();
            pair_sync(pair_bar);
            if (issuer) {
              tma_store_2d(&tmY, stage_buf, (w.nt * kBlockN + s * 64) * 2, w.row0 + quad * 32);
              bulk_commit();
            }
          }
        }
      }
      par ^= 1;
    }
    if (issuer) bulk_wait_all();                                // stores still read the staging buffer
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort) {
    if (tid == 0) atomicOr(p.status, static_cast<uint32_t>(TEMPO_STATUS_TIMEOUT));
    for (int i = 0; i < 50; ++i) __nanosleep(1000);  // let copies and MMAs in flight drain
  }
  if (warp == 1) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

size_t ffn_workspace_bytes(int M_cap) {
  return ((2 * sizeof(int32_t) * static_cast<size_t>(M_cap / kTileM)) + 255) & ~static_cast<size_t>(255);
}

cudaError_t launch_ffn(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmH, const CUtensorMap& tmY,
                       const FfnParams& p, int num_sms, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  const int grid = max(1, num_sms);   // one persistent CTA per SM; CTAs without work leave at once
  return launch_pdl(ffn_kernel, dim3(grid), dim3(kGemmThreads), kGemmSmemBytes, stream, tmA1, tmA2, tmH, tmY, p);
}

}  // namespace tempo
