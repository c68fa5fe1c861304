// Step 3 with CTA PAIRS (tcgen05 cta_group::2): an alternative to the one-CTA kernel, selected
// with tempo_set_ffn_mode(2).  Same results bit for bit; not the default.
//
// With many rows per instance the one-CTA kernel is bound by what one SM takes in: every
// 128x256x128 step needs 48 KB (A 16 KB + B 32 KB) and only four such stages fit in shared memory.
// Here two CTAs on neighbouring SMs (a cluster of two) compute a 256x256 tile together: each loads
// its own 128 rows of A and HALF of the B tile (128 of the 256 columns), the tensor cores of both
// SMs read both halves, and each SM accumulates its own 128 rows x 256 columns in its own tensor
// memory.  A step costs 32 KB of loads per SM and six stages fit.  Measured on B200 this is not
// faster (d = 8192, f = 1536, 8 instances x 2048 rows: 523 us against 505 us): with loads alone
// the pair kernel runs at 0.28 us per step, with MMAs alone at 0.37 us, together at 0.46 us - the
// half tile an SM reads from its neighbour appears to count against the same per-SM intake
// (about 110 KB/us) as its own loads, so the pair moves as many bytes per SM as the single CTA.
//
// Work items are (instance, 256-column tile, PAIR of M-tiles); the even CTA of the cluster (the
// leader) takes the pair's first M-tile, the odd CTA the second.  An instance with an odd number
// of M-tiles has one item whose second half is absent: the odd CTA then feeds its tensor core
// rows that exist (the leader's) and drops the result.
//
// Roles per CTA are those of the one-CTA kernel (384 threads: weight producer, MMA issuer,
// activation producer, scout, 8 epilogue warps) with these differences:
//   * all loads are TMA tensor copies with .cta_group::2, which lets the odd CTA's copies
//     complete on the LEADER's full barrier (weights and scale atoms through flat 128-byte-row
//     views of their buffers); the leader's producers announce the bytes of both CTAs;
//   * only the leader issues tcgen05.cp / tcgen05.mma (.cta_group::2); tcgen05.commit with
//     .multicast::cluster frees the stage / publishes the accumulator in both CTAs;
//   * the epilogue warps of both CTAs release the accumulator on the leader's barrier (remote
//     mbarrier arrive for the odd CTA).
// No load uses cluster multicast.  Every wait is bounded as in the one-CTA kernel.
#include "ffn_common.cuh"

namespace tempo {

constexpr int kPStages = 6;
constexpr int kPHalfB = kBBytes / 2;                        // 16 KB: this CTA's 128 columns of the B tile
constexpr int kPStageBytes = kABytes + kPHalfB;             // 32 KB
constexpr int kPSfBytes = kSfaBytes + kSfbBytes;            // 1536: own A atom + the whole B tile's two atoms
constexpr int kPThreads = 384;
constexpr int kPEpiWarp0 = 4;
constexpr size_t kPSmemBytes =
    static_cast<size_t>(kPStages) * (kPStageBytes + kPSfBytes) + 4 * kStoreBytes + 1024;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait on a barrier that the other CTA of the pair also arrives on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}
// TMA tensor copy into this CTA's shared memory whose bytes complete on a barrier that may live in
// the other CTA of the pair (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0,
                                                 int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(mask)
      : "memory");
}
__device__ __forceinline__ void tc_cp_sf_pair(uint32_t tmem_addr, uint64_t desc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(tmem_addr), "l"(desc) : "memory");
}
__device__ __forceinline__ void tc_mma_mxf8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
      : "memory");
}
// Instruction descriptor as in the one-CTA kernel, M = 256 (the pair's rows).
__device__ __forceinline__ uint32_t instr_desc_pair(int sf_id) {
  return (static_cast<uint32_t>(kBlockN >> 3) << 17) | (1u << 23) | (static_cast<uint32_t>(256 >> 4) << 24) |
         (static_cast<uint32_t>(sf_id) << 29) | (static_cast<uint32_t>(sf_id) << 4);
}

struct PairItem {
  int side;       // 0 gate/up, 1 down
  int inst, nt;
  int row0;       // first row of THIS CTA's M-tile (the leader's when this CTA's tile is absent)
  int present;    // this CTA's M-tile exists
  int m_tiles;    // M-tiles of the instance
};

// Pair-tiles before instance i: (M-tiles before i + instances before i with an odd count) / 2.
__device__ __forceinline__ int pairs_before(const int* toff, const uint16_t* odd, int i) {
  return (toff[i] + static_cast<int>(odd[i])) >> 1;
}

// Items of one side are numbered instance-major, then N-tile, then M-pair (as in the one-CTA kernel).
__device__ __forceinline__ PairItem decode_pair(int side, int x, const int* toff, const uint16_t* odd, int G, int NT,
                                                int rank) {
  int lo = 0, hi = G - 1;
  while (lo < hi) {                       // first i with NT * pairs_before(i+1) > x
    const int mid = (lo + hi) >> 1;
    if (NT * pairs_before(toff, odd, mid + 1) > x) hi = mid; else lo = mid + 1;
  }
  const int p0 = pairs_before(toff, odd, lo);
  const int local = x - NT * p0;
  const int Pi = pairs_before(toff, odd, lo + 1) - p0;
  const int Mi = toff[lo + 1] - toff[lo];
  const int mp = local % Pi;
  PairItem w;
  w.side = side;
  w.inst = lo;
  w.nt = local / Pi;
  w.m_tiles = Mi;
  const int mt = 2 * mp + rank;
  w.present = mt < Mi ? 1 : 0;
  w.row0 = (toff[lo] + (w.present ? mt : 2 * mp)) * kTileM;
  return w;
}

__global__ void __launch_bounds__(kPThreads, 1)
ffn_pair_kernel(const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmA2,
                const __grid_constant__ CUtensorMap tmY,
                const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmSfb,
                const __grid_constant__ CUtensorMap tmSfa1, const __grid_constant__ CUtensorMap tmSfa2,
                const FfnParams p, const PairRows pr) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t s_full[kPStages];
  __shared__ __align__(8) uint64_t s_empty[kPStages];
  __shared__ __align__(8) uint64_t s_acc_full;
  __shared__ __align__(8) uint64_t s_acc_empty;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort_storage;
  __shared__ int s_dep_storage;
  __shared__ int s_toff[kMaxSlots + 1];
  __shared__ uint16_t s_odd[kMaxSlots + 2];
  __shared__ float s_amax[2][2][kTileM];
  __shared__ int s_ok[2][4][2];
  volatile int* s_abort = &s_abort_storage;
  volatile int* s_dep = &s_dep_storage;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sf_base = smem_base + kPStages * kPStageBytes;
  const uint32_t store_base = sf_base + kPStages * kPSfBytes;
  const int G = p.G_max;
  const int rank = static_cast<int>(cluster_ctarank());
  const bool leader = rank == 0;
  pdl_trigger();
  if (tid == 0) {
    for (int s = 0; s < kPStages; ++s) { mbar_init(smem_u32(&s_full[s]), 2); mbar_init(smem_u32(&s_empty[s]), 1); }
    mbar_init(smem_u32(&s_acc_full), 1);
    mbar_init(smem_u32(&s_acc_empty), 16);                  // 8 epilogue warps of each CTA
    s_abort_storage = 0;
    s_dep_storage = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA1)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA2)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmW)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmSfb)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmSfa1)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmSfa2)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
  }
  if (warp == 1) {   // both CTAs of the pair take part in the allocation
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  pdl_wait();
  const int m_pad = max(0, min(*p.m_pad, p.M_cap)) & ~(kTileM - 1);
  for (int i = tid; i <= G; i += kPThreads) s_toff[i] = max(0, min(p.inst_off[i], m_pad)) >> 7;
  __syncthreads();
  if (warp == 0) {   // odd[i] = instances before i with an odd number of M-tiles
    int carry = 0;
    for (int base = 0; base < G; base += 32) {
      const int i = base + lane;
      const int is_odd = i < G ? ((s_toff[i + 1] - s_toff[i]) & 1) : 0;
      int incl = is_odd;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (i < G) s_odd[i] = static_cast<uint16_t>(carry + incl - is_odd);
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_odd[G] = static_cast<uint16_t>(carry);
  }
  tc_fence_before();
  cluster_sync_all();          // barriers and tensor memory of both CTAs are ready; also a CTA barrier
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  const int n_pairs = pairs_before(s_toff, s_odd, G);
  const int n1 = (p.run_mask & 1) ? n_pairs * p.side[0].NT : 0;
  const int n2 = (p.run_mask & 2) ? n_pairs * p.side[1].NT : 0;
  const bool fused = p.run_mask == 3;
  const int Kb1 = p.side[0].Kb, Kb2 = p.side[1].Kb;
  const int cid = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

  // the leader's barriers as the odd CTA must address them (its own for the leader itself)
  const uint32_t full0_leader = map_to_cta(smem_u32(&s_full[0]), 0);
  const uint32_t acc_empty_leader = map_to_cta(smem_u32(&s_acc_empty), 0);

  if (warp == 0) {
    // ------------------------------- weight producer ------------------------------------------
    // This CTA's half of every B tile: rows [128*rank, +128) of the packed 256-row tile, and the
    // tile's two scale atoms (both CTAs need all 256 columns' scales).
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      TileIter it(cid, n_clusters, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const GemmSide& gs = p.side[side];
        const PairItem w = decode_pair(side, x, s_toff, s_odd, G, gs.NT, rank);
        const uint32_t tile = static_cast<uint32_t>(w.inst) * gs.NT + w.nt;
        const uint32_t wrow = pr.w_row[side] + tile * gs.Kb * 256u + static_cast<uint32_t>(rank) * 128u;
        const uint32_t sfrow = pr.sfb_row[side] + tile * gs.JK * 8u;
        for (int kb = 0; kb < gs.Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort)) { ok = false; break; }
          const uint32_t sB = smem_base + stage * kPStageBytes + kABytes;
          const uint32_t sSfb = sf_base + stage * kPSfBytes + kSfaBytes;
          const bool with_sf = (kb & 3) == 0;
          if (leader) mbar_arrive_expect_tx(smem_u32(&s_full[stage]), 2 * kPHalfB + (with_sf ? 2 * kSfbBytes : 0));
          const uint32_t full = full0_leader + stage * 8u;
          tma_load_2d_pair(sB, &tmW, full, 0, static_cast<int>(wrow + kb * 256u));
          if (with_sf) tma_load_2d_pair(sSfb, &tmSfb, full, 0, static_cast<int>(sfrow + (kb >> 2) * 8u));
          if (++stage == kPStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------- activation producer --------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      int n_down = 0;
      bool ok = true;
      TileIter it(cid, n_clusters, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const GemmSide& gs = p.side[side];
        const PairItem w = decode_pair(side, x, s_toff, s_odd, G, gs.NT, rank);
        const CUtensorMap* tm = side == 0 ? &tmA1 : &tmA2;
        const CUtensorMap* tsf = side == 0 ? &tmSfa1 : &tmSfa2;
        const uint32_t sfa_row = static_cast<uint32_t>(w.row0 >> 7) * gs.JK * 4u;
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
          __threadfence_block();
          asm volatile("fence.proxy.async;" ::: "memory");   // H was written by ordinary stores, TMA reads it
        }
        for (int kb = 0; kb < gs.Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort)) { ok = false; break; }
          const uint32_t sA = smem_base + stage * kPStageBytes;
          const uint32_t sSfa = sf_base + stage * kPSfBytes;
          const bool with_sf = (kb & 3) == 0;
          if (leader) mbar_arrive_expect_tx(smem_u32(&s_full[stage]), 2 * kABytes + (with_sf ? 2 * kSfaBytes : 0));
          const uint32_t full = full0_leader + stage * 8u;
          tma_load_2d_pair(sA, tm, full, kb * kBlockK, w.row0);
          if (with_sf) tma_load_2d_pair(sSfa, tsf, full, 0, static_cast<int>(sfa_row + (kb >> 2) * 4u));
          if (++stage == kPStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------- dependency scout -----------------------------------------
    // As in the one-CTA kernel, for this CTA's own M-tile of every down item; an absent tile has
    // nothing to wait for.
    if (lane == 0 && fused) {
      TileIter it(cid, n_clusters, n1, n2, Kb1, Kb2);
      int side, x, cleared = 0;
      const int want = 4 * p.side[0].NT;
      bool ok = true;
      while (ok && it.next(side, x)) {
        if (side == 0) continue;
        const PairItem w = decode_pair(1, x, s_toff, s_odd, G, p.side[1].NT, rank);
        if (!w.present) { *s_dep = ++cleared; continue; }
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
        __threadfence_block();
        *s_dep = ++cleared;                      // tell the producer first, then do the bookkeeping
        if (atomicAdd(p.done + tau, 1) == p.side[1].NT - 1) {
          atomicExch(p.ready + tau, 0);
          atomicExch(p.done + tau, 0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) ------------------------------
    if (leader && lane == 0) {
      uint32_t stage = 0, phase = 0, acc_phase = 0;
      bool ok = true;
      TileIter it(cid, n_clusters, n1, n2, Kb1, Kb2);
      int side, x;
      while (ok && it.next(side, x)) {
        const int Kb = p.side[side].Kb;
        if (!mbar_wait_cluster(smem_u32(&s_acc_empty), acc_phase ^ 1u, s_abort)) break;
        tc_fence_after();
        for (int kb = 0; kb < Kb; ++kb) {
          if (!mbar_wait(smem_u32(&s_full[stage]), phase, s_abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sA = smem_base + stage * kPStageBytes, sB = sA + kABytes;
          const uint32_t sSF = sf_base + stage * kPSfBytes;
          const uint32_t sfa_t = tmem_base + kSfCol0 + 16u * ((kb >> 2) & 1);
          const uint32_t sfb_t = sfa_t + 4;
          if ((kb & 3) == 0) {
            tc_cp_sf_pair(sfa_t, smem_desc_sf(sSF));
            tc_cp_sf_pair(sfb_t, smem_desc_sf(sSF + kSfaBytes));
            tc_cp_sf_pair(sfb_t + 4, smem_desc_sf(sSF + kSfaBytes + 512));
          }
          const uint32_t idesc = instr_desc_pair(kb & 3);
          const uint64_t da = smem_desc_sw128(sA), db = smem_desc_sw128(sB);
#pragma unroll
          for (int ks = 0; ks < kBlockK / 32; ++ks)
            tc_mma_mxf8_pair(tmem_base, da + 2u * ks, db + 2u * ks, idesc, sfa_t, sfb_t, (kb | ks) != 0 ? 1u : 0u);
          tc_commit_pair(smem_u32(&s_empty[stage]));
          if (++stage == kPStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit_pair(smem_u32(&s_acc_full));
        acc_phase ^= 1u;
      }
    }
  } else if (warp >= kPEpiWarp0) {
    // ------------------------------- epilogue --------------------------------------------------
    // As in the one-CTA kernel (two warps per tensor-memory lane quadrant, raw copy to registers,
    // release, arithmetic, ordinary stores for H, swizzled staging + TMA stores for Y), on this
    // CTA's own 128 rows.
    const int quad = warp & 3;
    const int half = (warp - kPEpiWarp0) >> 2;
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const uint32_t stage_buf = store_base + quad * kStoreBytes;
    const uint32_t my_line = stage_buf + lane * 128;
    const bool issuer = half == 0 && lane == 0;
    const int pair_bar = 1 + quad;
    const int r_in_tile = quad * 32 + lane;
    uint32_t acc_phase = 0;
    int par = 0;
    TileIter it(cid, n_clusters, n1, n2, Kb1, Kb2);
    int side, x;
    while (it.next(side, x)) {
      const PairItem w = decode_pair(side, x, s_toff, s_odd, G, p.side[side].NT, rank);
      const int row = w.row0 + r_in_tile;
      const bool ok = mbar_wait(smem_u32(&s_acc_full), acc_phase, s_abort);
      acc_phase ^= 1u;
      if (lane == 0) s_ok[par][quad][half] = ok ? 1 : 0;
      pair_sync(pair_bar);
      if (!(s_ok[par][quad][0] && s_ok[par][quad][1])) break;
      tc_fence_after();
      if (!w.present) {
        // nothing of this CTA's accumulator is wanted: hand it back at once
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
      } else if (side == 0) {
        uint32_t g[2][32], u[2][32];
        tmem_ld32(taddr + half * 64, g[0]);
        tmem_ld32(taddr + half * 64 + 32, g[1]);
        tmem_ld32(taddr + 128 + half * 64, u[0]);
        tmem_ld32(taddr + 128 + half * 64 + 32, u[1]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
        pin32(g[0]); pin32(g[1]); pin32(u[0]); pin32(u[1]);
        float amax = 0.f;
        // A row whose gate values are all zero (a padding row: its activations are zero) gives
        // H = 0 whatever `up` holds; with few live rows per tile most rows are like that, and
        // skipping their exponentials shortens the wait of the down tiles that need this H block.
        // H overwrites the gate registers (an all-zero gate row already is its own H).
        uint32_t any_gate = 0;
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i) any_gate |= g[c][i];
        if ((any_gate & 0x7fffffffu) != 0) {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float gv = __uint_as_float(g[c][i]), uv = __uint_as_float(u[c][i]);
              const float hv = __fdividef(gv, 1.f + __expf(-gv)) * uv;
              g[c][i] = __float_as_uint(hv);
              amax = fmaxf(amax, fabsf(hv));
            }
          }
        }
#define TEMPO_H(j) __uint_as_float(g[(j) >> 5][(j) & 31])
        s_amax[par][half][r_in_tile] = amax;
        pair_sync(pair_bar);
        amax = fmaxf(amax, s_amax[par][half ^ 1][r_in_tile]);
        const int eps = pow2_scale_exponent(amax);
        const float inv = pow2_neg(eps);
        // ordinary stores for H, as in the one-CTA kernel (a TMA store would queue behind the loads)
        uint4* dst = reinterpret_cast<uint4*>(p.h_q + static_cast<size_t>(row) * p.f + w.nt * 128 + half * 64);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 q;
          q.x = cvt_e4m3x4(TEMPO_H(16 * v + 0) * inv, TEMPO_H(16 * v + 1) * inv, TEMPO_H(16 * v + 2) * inv, TEMPO_H(16 * v + 3) * inv);
          q.y = cvt_e4m3x4(TEMPO_H(16 * v + 4) * inv, TEMPO_H(16 * v + 5) * inv, TEMPO_H(16 * v + 6) * inv, TEMPO_H(16 * v + 7) * inv);
          q.z = cvt_e4m3x4(TEMPO_H(16 * v + 8) * inv, TEMPO_H(16 * v + 9) * inv, TEMPO_H(16 * v + 10) * inv, TEMPO_H(16 * v + 11) * inv);
          q.w = cvt_e4m3x4(TEMPO_H(16 * v + 12) * inv, TEMPO_H(16 * v + 13) * inv, TEMPO_H(16 * v + 14) * inv, TEMPO_H(16 * v + 15) * inv);
          dst[v] = q;
        }
#undef TEMPO_H
        if (half == 0) p.h_sf[sf_index(row, w.nt, p.J_h)] = static_cast<uint8_t>(eps + 127);
        if (fused) {                                           // publish these 32 rows of the H block
          pair_sync(pair_bar);
          if (issuer) {
            __threadfence();
            atomicAdd(p.ready + (w.row0 >> 7), 1);
          }
        }
      } else {
        uint32_t a[4][32];
#pragma unroll
        for (int s = 0; s < 4; ++s) tmem_ld32(taddr + s * 64 + half * 32, a[s]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
        pin32(a[0]); pin32(a[1]); pin32(a[2]); pin32(a[3]);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          if (w.nt * kBlockN + s * 64 < p.d) {
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
    if (issuer) bulk_wait_all();
    __syncwarp();
  }

  // Neither CTA may leave (or free tensor memory) while the other still reads its shared memory
  // or writes its accumulator.
  tc_fence_before();
  cluster_sync_all();
  if (*s_abort) {
    if (tid == 0) atomicOr(p.status, static_cast<uint32_t>(TEMPO_STATUS_TIMEOUT));
    for (int i = 0; i < 50; ++i) __nanosleep(1000);  // let copies and MMAs in flight drain
  }
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

cudaError_t launch_ffn_pair(const PairMaps& m, const FfnParams& p, const PairRows& pr, int num_sms, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(ffn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kPSmemBytes));
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * max(1, num_sms / 2));   // one persistent CTA pair per two SMs
  cfg.blockDim = dim3(kPThreads);
  cfg.dynamicSmemBytes = kPSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // Down items wait for gate/up items of other pairs, so every pair of the grid must be resident.
  int resident = 0;
  e = cudaOccupancyMaxActiveClusters(&resident, ffn_pair_kernel, &cfg);
  if (e != cudaSuccess) return e;
  if (resident < 1) return cudaErrorLaunchOutOfResources;
  if (static_cast<unsigned int>(2 * resident) < cfg.gridDim.x) cfg.gridDim = dim3(2 * resident);
  return cudaLaunchKernelEx(&cfg, ffn_pair_kernel, m.a1, m.a2, m.y, m.w, m.sfb, m.sfa1, m.sfa2, p, pr);
}

}  // namespace tempo
