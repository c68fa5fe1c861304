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
//              shared memory).  Y leaves through swizzled staging in shared memory and TMA tensor
//              stores; H leaves through ordinary 16-byte stores, because other CTAs wait for it and
//              a TMA store queues behind the weight loads already issued for the next tile
// Scales are UE8M0 per 128 K-elements; the MMA takes one scale byte per row (A) and per column
// (B) for each K=32 step, so the four steps of a K-block select the same byte (scale id kb % 4).
//
// Every wait is bounded: after FfnParams::wait_ns the CTA raises an abort flag, all roles leave their
// loops, TEMPO_STATUS_TIMEOUT is set and tensor memory is freed.
#include "ffn_common.cuh"

namespace tempo {

constexpr int kStages = 4;
constexpr int kStageBytes = kABytes + kBBytes + 2048;     // 51200, a multiple of 1024
constexpr int kGemmThreads = 384;
constexpr int kEpiWarp0 = 4;                               // first of the 8 epilogue warps
constexpr int kGatherWarp0 = 12;                           // gather form: 4 more warps, one per stage of the ring
constexpr int kGatherThreads = 512;
constexpr size_t kGemmSmemBytes = static_cast<size_t>(kStages) * kStageBytes + 4 * kStoreBytes + 1024;

// kBf16 = false: the fp8 path described above.  kBf16 = true: the bf16 variant (the paper calibrates a
// bf16 grouped GEMM beside the fp8 one, Section 2.1): the same ring, roles and tiles with 64 bf16
// values per 128-byte K-block, tcgen05.mma.kind::f16 without scales, and H stored as bf16.
//
// kGather = true (fp8 only): the gate/up operand is not read from a permuted copy.  Four more warps
// (12-15) fetch each row of the A tile from the per-token quantised activations x_q by the row's
// token (row_pair / k) with 16-byte cp.async copies straight into the 128-byte-swizzled stage, and its
// scale bytes from x_sf into the stage's scale atom; rows without a pair are zero-filled.  That takes
// the permuted a_q / a_sf buffers (one write and NT re-reads of every row) out of the block.  Each
// gather warp owns one stage of the ring and is that stage's second arrival on gate/up tiles, as the
// activation producer is on down tiles.  512 threads leave 128 registers per thread at launch; the
// producer and gather warps hand most of theirs to the epilogue warps (setmaxnreg).  Measured on B200 this
// form's kernel is 15-25 % slower than the permuted form's (the tensor pipe waits for A rows that 16-byte
// copies deliver later than one bulk tensor copy would): it is for callers who want the memory of the
// permuted copy back, not for speed.
template <bool kBf16, bool kGather>
__global__ void __launch_bounds__(kGather ? kGatherThreads : kGemmThreads, 1)
ffn_kernel(const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmA2,
           const __grid_constant__ CUtensorMap tmY, const FfnParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t s_full[kStages];
  __shared__ __align__(8) uint64_t s_empty[kStages];
  __shared__ __align__(8) uint64_t s_acc_full;
  __shared__ __align__(8) uint64_t s_acc_empty;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort_storage;
  __shared__ int s_dep_storage;
  __shared__ int s_toff[kMaxSlots + 1];
  __shared__ uint16_t s_cold[kMaxSlots + 2];   // M-tiles of cold instances before each instance (at most 2 each)
  __shared__ float s_amax[2][2][kTileM];   // [tile parity][column half][row]: row maxima of the two half-row warps
  __shared__ int s_ok[2][4][2];             // [tile parity][quadrant][column half]: that warp's wait succeeded
  volatile int* s_abort = &s_abort_storage;
  volatile int* s_dep = &s_dep_storage;   // down tiles of this CTA whose H rows are known complete

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int G = p.G_max;
  const unsigned long long wait_ns = p.wait_ns;
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
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();
  const int stride = p.stride_tiles;
  if (stride > 0) {
    // masked layout: M-tiles in use before each instance, from the row counts (warp 0 scans)
    if (warp == 0) {
      int carry = 0;
#pragma unroll 1
      for (int base = 0; base < G; base += 32) {
        const int i = base + lane;
        const int c = i < G ? min(stride, (max(0, p.inst_count[i]) + kTileM - 1) / kTileM) : 0;
        int incl = c;
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        if (i < G) s_toff[i] = carry + incl - c;
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) s_toff[G] = carry;
    }
  } else {
    const int m_pad_c = max(0, min(*p.m_pad, p.M_cap)) & ~(kTileM - 1);
#pragma unroll 1
    for (int i = tid; i <= G; i += static_cast<int>(blockDim.x)) s_toff[i] = max(0, min(p.inst_off[i], m_pad_c)) >> 7;
  }
  __syncthreads();
  const int m_tiles = s_toff[G];
  const int n1 = (p.run_mask & 1) ? m_tiles * p.side[0].NT : 0;
  const int n2 = (p.run_mask & 2) ? m_tiles * p.side[1].NT : 0;
  const bool fused = p.run_mask == 3;
  const int Kb1 = p.side[0].Kb, Kb2 = p.side[1].Kb;
  if (warp == 0) {   // cold[i] = M-tiles of cold instances before instance i
    int carry = 0;
#pragma unroll 1
    for (int base = 0; base < G; base += 32) {
      const int i = base + lane;
      const int Mi = i < G ? s_toff[i + 1] - s_toff[i] : 0;
      const int c = Mi <= kColdTiles ? Mi : 0;
      int incl = c;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (i < G) s_cold[i] = static_cast<uint16_t>(carry + incl - c);
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_cold[G] = static_cast<uint16_t>(carry);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  const int cold_tiles = s_cold[G], hot_tiles = m_tiles - cold_tiles;
  const TileOrder order1(p.side[0].NT, hot_tiles, cold_tiles, gridDim.x), order2(p.side[1].NT, hot_tiles, cold_tiles, gridDim.x);
  // Roles by warpgroup (the register hand-over of the gather form works on whole warpgroups of four warps):
  // 128 x (72 + 176 + 176 + 80) = 64512 of the SM's 65536 registers.
  if (warp < kEpiWarp0) {
    if constexpr (kGather) asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0) {
      // ------------------------------- weight producer ------------------------------------------
      if (lane == 0) {
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
        int side, x;
        while (ok && it.next(side, x)) {
          const GemmSide& gs = p.side[side];
          const WorkItem w = decode_item(side, x, s_toff, s_cold, G, side == 0 ? order1 : order2, stride);
          const uint8_t* sfb_src = gs.sfb + (static_cast<size_t>(w.inst) * gs.NT + w.nt) * gs.JK * kSfbBytes;
          const uint8_t* b_src = gs.wt + (static_cast<size_t>(w.inst) * gs.NT + w.nt) * gs.Kb * kBBytes;
          const bool stream_b = w.m_tiles <= 2;
#pragma unroll 1
          for (int kb = 0; kb < gs.Kb; ++kb) {
            if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort, wait_ns)) { ok = false; break; }
            const uint32_t full = smem_u32(&s_full[stage]);
            const uint32_t sB = smem_base + stage * kStageBytes + kABytes, sSF = sB + kBBytes;
            const bool with_sf = !kBf16 && (kb & 3) == 0;
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
          const WorkItem w = decode_item(side, x, s_toff, s_cold, G, side == 0 ? order1 : order2, stride);
          const uint8_t* sfa_src = gs.sfa + static_cast<size_t>(w.row0 >> 7) * gs.JK * kSfaBytes;
          const CUtensorMap* tm = side == 0 ? &tmA1 : &tmA2;
          if (kGather && side == 0) {
            // The gather warps fill these stages.  This thread still follows the ring slot by slot: an
            // mbarrier wait tells one phase from the next only, so a waiter that jumped several phases
            // ahead would take a stage that is still in use for a free one.
#pragma unroll 1
            for (int kb = 0; kb < gs.Kb; ++kb) {
              if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort, wait_ns)) { ok = false; break; }
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            continue;
          }
          if (side == 1 && fused) {
            // wait until the scout (warp 3) has seen every H block of these 128 rows complete
            ++n_down;
            unsigned long long t0 = 0;
            for (uint32_t spin = 0; *s_dep < n_down; ++spin) {
              if ((spin & 255u) == 255u) {
                if (*s_abort) { ok = false; break; }
                const unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > wait_ns) { *s_abort = 1; ok = false; break; }
              }
            }
            if (!ok) break;
            // The scout's acquire load saw the rows published; its word reaches this thread through
            // shared memory (block-scope fences on both sides), then the proxy fence orders the
            // ordinary stores that wrote H before the TMA reads below.
            __threadfence_block();
            asm volatile("fence.proxy.async;" ::: "memory");
          }
#pragma unroll 1
          for (int kb = 0; kb < gs.Kb; ++kb) {
            if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, s_abort, wait_ns)) { ok = false; break; }
            const uint32_t full = smem_u32(&s_full[stage]);
            const uint32_t sA = smem_base + stage * kStageBytes, sSF = sA + kABytes + kBBytes;
            const bool with_sf = !kBf16 && (kb & 3) == 0;
            mbar_arrive_expect_tx(full, kABytes + (with_sf ? kSfaBytes : 0));
            tma_load_2d(sA, tm, full, kb * kBlockK, w.row0);
            if (with_sf) bulk_load(sSF, sfa_src + static_cast<size_t>(kb >> 2) * kSfaBytes, kSfaBytes, full);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    } else if (warp == 3) {
      // ------------------------------- dependency scout -----------------------------------------
      // Runs ahead through this CTA's down tiles: waits (bounded) until the four epilogue warp pairs of
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
          const WorkItem w = decode_item(1, x, s_toff, s_cold, G, order2, stride);
          const int tau = w.row0 >> 7;
          unsigned long long t0 = 0;
          for (uint32_t spin = 0; ld_acquire(p.ready + tau) < want; ++spin) {
            if ((spin & 63u) == 63u) {
              if (*s_abort) { ok = false; break; }
              const unsigned long long now = global_timer_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > wait_ns) { *s_abort = 1; ok = false; break; }
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
      // ------------------------------- MMA issuer -----------------------------------------------
      if (lane == 0) {
        uint32_t stage = 0, phase = 0, acc_phase = 0;
        bool ok = true;
        TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
        int side, x;
        while (ok && it.next(side, x)) {
          const int Kb = p.side[side].Kb;
          if (!mbar_wait(smem_u32(&s_acc_empty), acc_phase ^ 1u, s_abort, wait_ns)) break;
          tc_fence_after();
#pragma unroll 1
          for (int kb = 0; kb < Kb; ++kb) {
            if (!mbar_wait(smem_u32(&s_full[stage]), phase, s_abort, wait_ns)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sA = smem_base + stage * kStageBytes, sB = sA + kABytes, sSF = sB + kBBytes;
            const uint32_t sfa_t = tmem_base + kSfCol0 + 16u * ((kb >> 2) & 1);
            const uint32_t sfb_t = sfa_t + 4;
            const uint64_t da = smem_desc_sw128(sA), db = smem_desc_sw128(sB);
            if constexpr (kBf16) {
#pragma unroll
              for (int ks = 0; ks < kBlockK / 32; ++ks)     // 16 bf16 values = 32 bytes per instruction
                tc_mma_bf16(tmem_base, da + 2u * ks, db + 2u * ks, instr_desc_bf16(), (kb | ks) != 0 ? 1u : 0u);
            } else {
              if ((kb & 3) == 0) {
                tc_cp_sf(sfa_t, smem_desc_sf(sSF));
                tc_cp_sf(sfb_t, smem_desc_sf(sSF + kSfaBytes));
                tc_cp_sf(sfb_t + 4, smem_desc_sf(sSF + kSfaBytes + 512));
              }
              const uint32_t idesc = instr_desc(kb & 3);
#pragma unroll
              for (int ks = 0; ks < kBlockK / 32; ++ks)
                tc_mma_mxf8(tmem_base, da + 2u * ks, db + 2u * ks, idesc, sfa_t, sfb_t, (kb | ks) != 0 ? 1u : 0u);
            }
            tc_commit(smem_u32(&s_empty[stage]));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) tc_commit(smem_u32(&s_acc_full));
          acc_phase ^= 1u;
        }
      }
    }
  } else if (kGather && warp >= kGatherWarp0) {
    if constexpr (kGather) asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
    // ------------------------------- row gather (gate/up operand) -------------------------------
    // Each of the four warps owns ONE stage of the ring (warp gw takes every K-block that lands in stage gw)
    // and copies all 128 rows of its K-block: a lane copies the 16-byte chunk (lane & 7) of 32 rows, so one
    // instruction of the warp covers four whole 128-byte rows.  It then waits for its own copies, makes them
    // visible to the tensor core's reads (async proxy) and arrives on the stage's barrier; meanwhile the other
    // three warps have their K-blocks in flight, so four stages of activations are under way at once, as
    // with the tensor copies of the permuted form.  On down tiles the warp only follows its stage's phases:
    // an mbarrier wait tells one phase from the next only, so nobody may skip ahead.
    static_assert(kStages == 4, "one gather warp per stage");
    const int gw = warp - kGatherWarp0;
    const int chunk = lane & 7, sub = lane >> 3;
    const int kshift = (p.k & (p.k - 1)) == 0 ? __ffs(p.k) - 1 : -1;
    const uint32_t d16 = static_cast<uint32_t>(p.d) >> 4;          // row pitch of x_q in 16-byte units
    const uint4* xq16 = reinterpret_cast<const uint4*>(p.x_q);
    const uint32_t my_empty = smem_u32(&s_empty[gw]), my_full = smem_u32(&s_full[gw]);
    const uint32_t sA = smem_base + gw * kStageBytes, sSF = sA + kABytes + kBBytes;
    uint32_t phase = 0;
    uint32_t cnt = 0;                                              // K-blocks of this CTA so far (stage = cnt % 4)
    bool ok = true;
    TileIter it(blockIdx.x, gridDim.x, n1, n2, Kb1, Kb2);
    int side, x;
    while (ok && it.next(side, x)) {
      const int Kb = p.side[side].Kb;
      // first K-block of this tile in my stage, and how many of them
      int kb = static_cast<int>((static_cast<uint32_t>(gw) - cnt) & (kStages - 1));
      cnt += static_cast<uint32_t>(Kb);
      if (side == 1) {
#pragma unroll 1
        for (; kb < Kb; kb += kStages) {
          if (!mbar_wait(my_empty, phase ^ 1u, s_abort, wait_ns)) { ok = false; break; }
          phase ^= 1u;
        }
        continue;
      }
      const WorkItem w = decode_item(0, x, s_toff, s_cold, G, order1, stride);
      // x_q offset (16-byte units) of each of this lane's 32 rows; ~0: a row without a pair, zero-filled
      uint32_t off16[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int pr = __ldg(p.row_pair + w.row0 + i * 4 + sub);
        const int t = min(kshift >= 0 ? pr >> kshift : pr / p.k, p.T - 1);
        off16[i] = pr < 0 ? 0xffffffffu : static_cast<uint32_t>(t) * d16 + chunk;
      }
      // scale atom: this lane supplies the 4-byte word of rows lane, lane + 32, lane + 64, lane + 96
      int t_sf[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int pr = __ldg(p.row_pair + w.row0 + q * 32 + lane);
        t_sf[q] = pr < 0 ? -1 : min(kshift >= 0 ? pr >> kshift : pr / p.k, p.T - 1);
      }
#pragma unroll 1
      for (; kb < Kb; kb += kStages) {
        if (!mbar_wait(my_empty, phase ^ 1u, s_abort, wait_ns)) { ok = false; break; }
        phase ^= 1u;
        const uint32_t kb16 = static_cast<uint32_t>(kb) * (kBlockK / 16);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int r = i * 4 + sub;
          const uint32_t dst = sA + r * 128 + ((chunk ^ (r & 7)) << 4);
          const bool live = off16[i] != 0xffffffffu;
          cp_async_16(dst, xq16 + (live ? off16[i] + kb16 : 0u), live ? 16u : 0u);
        }
        if ((kb & 3) == 0) {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            cp_async_4(sSF + lane * 16 + q * 4,
                       p.x_sf + (t_sf[q] < 0 ? 0 : static_cast<size_t>(t_sf[q]) * p.x_sf_stride + kb), t_sf[q] < 0 ? 0u : 4u);
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(my_full);
      }
    }
  } else {
    if constexpr (kGather) asm volatile("setmaxnreg.inc.sync.aligned.u32 176;");
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
      const WorkItem w = decode_item(side, x, s_toff, s_cold, G, side == 0 ? order1 : order2, stride);
      const int row = w.row0 + r_in_tile;
      // Both warps of a pair must take the same way out: they vote on the outcome of the wait.
      const bool ok = mbar_wait(smem_u32(&s_acc_full), acc_phase, s_abort, wait_ns);
      acc_phase ^= 1u;
      if (lane == 0) s_ok[par][quad][half] = ok ? 1 : 0;
      pair_sync(pair_bar);
      if (!(s_ok[par][quad][0] && s_ok[par][quad][1])) break;
      tc_fence_after();
      if (side == 0 && kBf16) {
        // H columns [64*s + 32*half, +32), s = 0, 1: gate from the same accumulator columns, up 128
        // columns further on; H leaves as bf16, 64 bytes of the row per thread and step.
        uint32_t g[2][32], u[2][32];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          tmem_ld32(taddr + s * 64 + half * 32, g[s]);
          tmem_ld32(taddr + 128 + s * 64 + half * 32, u[s]);
        }
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_acc_empty));
        pin32(g[0]); pin32(g[1]); pin32(u[0]); pin32(u[1]);
        uint32_t any_gate = 0;                               // all-zero gate row (padding): H = 0, skip the exponentials
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
          for (int i = 0; i < 32; ++i) any_gate |= g[s][i];
        const bool live_row = (any_gate & 0x7fffffffu) != 0;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) packed[i] = 0;
          if (live_row) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float g0 = __uint_as_float(g[s][2 * i]), g1 = __uint_as_float(g[s][2 * i + 1]);
              const float h0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(u[s][2 * i]);
              const float h1 = __fdividef(g1, 1.f + __expf(-g1)) * __uint_as_float(u[s][2 * i + 1]);
              const __nv_bfloat162 b = __floats2bfloat162_rn(h0, h1);
              packed[i] = *reinterpret_cast<const uint32_t*>(&b);
            }
          }
          // ordinary stores, as for the fp8 H (a TMA store would queue behind the next tile's weight loads)
          uint4* dst = reinterpret_cast<uint4*>(p.h_q + (static_cast<size_t>(row) * p.f + w.nt * 128 + s * 64 + half * 32) * 2);
#pragma unroll
          for (int v = 0; v < 4; ++v) dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
        }
        if (fused) {                                           // publish these 32 rows of the H block
          pair_sync(pair_bar);
          if (issuer) {
            __threadfence();
            atomicAdd(p.ready + (w.row0 >> 7), 1);
          }
        }
      } else if (side == 0) {
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
        // H goes out with ordinary 16-byte stores (64 bytes of the row per thread), not through the
        // TMA unit: there a store queues behind the weight loads already issued for the next tile,
        // which held the H block back by 4-9 us while down tiles of other CTAs waited for it.
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
        if (fused) {                                           // publish these 32 rows of the H block:
          pair_sync(pair_bar);                                 // both warps' stores are issued, then one
          if (issuer) {                                        // thread fences for the pair and bumps the counter
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

template <bool kBf16, bool kGather>
static cudaError_t launch_ffn_t(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmY,
                                const FfnParams& p, int num_sms, cudaStream_t stream) {
  static std::atomic<unsigned long long> smem_set{0};
  cudaError_t e = smem_limit_once(ffn_kernel<kBf16, kGather>, kGemmSmemBytes, smem_set);
  if (e != cudaSuccess) return e;
  const int grid = max(1, num_sms);   // one persistent CTA per SM; CTAs without work leave at once
  return launch_pdl(ffn_kernel<kBf16, kGather>, dim3(grid), dim3(kGather ? kGatherThreads : kGemmThreads), kGemmSmemBytes,
                    stream, tmA1, tmA2, tmY, p);
}

cudaError_t launch_ffn(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmY,
                       const FfnParams& p, int num_sms, cudaStream_t stream) {
  return launch_ffn_t<false, false>(tmA1, tmA2, tmY, p, num_sms, stream);
}

cudaError_t launch_ffn_gather(const CUtensorMap& tmA2, const CUtensorMap& tmY, const FfnParams& p, int num_sms,
                              cudaStream_t stream) {
  return launch_ffn_t<false, true>(tmA2, tmA2, tmY, p, num_sms, stream);   // the first map is never used
}

cudaError_t launch_ffn_bf16(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmY,
                            const FfnParams& p, int num_sms, cudaStream_t stream) {
  return launch_ffn_t<true, false>(tmA1, tmA2, tmY, p, num_sms, stream);
}

}  // namespace tempo
