// Step 1: fused count + quota dispatch + padded grouped layout, one launch of one thread-block cluster.
//
// The paper's in-graph contract (Section 4.4): dispatch through the replica table fused with
// count collection into a cumulative per-expert counter, CUDA-graph padding rows masked, rows
// renormalised at use, zero-sum row -> uniform over the replicas holding the expert.  Here the
// table holds integer shares x_{e,r} (Eq. 2) that are honoured exactly and deterministically:
// pairs of one expert are ranked by ascending pair index and cut into contiguous rank runs.
//
// Ranks come from scans, not from atomics, so the result is bit-reproducible:
//   pass 1  the live pairs are cut into contiguous chunks, one per CTA of the cluster, and inside
//           a CTA into one contiguous range per warp; every warp builds its own histogram
//           (ballots over the id bits group equal experts inside a 32-pair step);
//   scan    per expert, an exclusive prefix over the 32 warp histograms, then over the CTAs of the
//           cluster (each CTA reads the others' totals through distributed shared memory), gives
//           every warp's base rank and the total n_e; the replica boundaries B_r, the rows of
//           each instance and the padded offsets follow from the quota row (every CTA computes
//           them, CTA 0 writes them out);
//   pass 2  every warp walks its range again, rank = base + position among equal lanes, and
//           scatters pair -> row and row -> pair.
// The cluster barriers are hardware barriers: nothing spins.
//
// The kernel runs once through a long body on one to eight SMs, so it pays for every instruction line it has
// to fetch: the loops outside the two passes are kept rolled (#pragma unroll 1), which takes the code from 57 KB
// to 23 KB and 0.8 us off a decode-sized launch.
#include <cooperative_groups.h>

#include "dispatch_common.cuh"

namespace cg = cooperative_groups;

namespace tempo {

__global__ void __launch_bounds__(kDispThreads, 1) count_dispatch_kernel(const DispatchParams p) {
  extern __shared__ int32_t smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int NC = static_cast<int>(cluster.num_blocks());
  const int cta = static_cast<int>(cluster.block_rank());
  const int E = p.E, R = p.R_max, G = p.G_max;
  int32_t* hist = smem;                       // [kDispWarps][E]  warp histograms -> exclusive bases inside the CTA
  int32_t* tot = hist + kDispWarps * E;       // [E]              this CTA's totals (read by the other CTAs)
  int32_t* cbase = tot + E;                   // [E]              pairs of the expert in lower-ranked CTAs
  int32_t* bnd = cbase + E;                   // [E][R]           cumulative rank boundaries B_r
  int32_t* owner = bnd + E * R;               // [G]              first (e,r) entry naming the slot
  int32_t* m_inst = owner + G;                // [G]              rows of each instance
  int32_t* off = m_inst + G;                  // [G+1]            padded offsets (not clamped)
  int32_t* rmap_s = off + G + 1;              // [E][R]           replica_map, staged once
  int32_t* quota_s = rmap_s + E * R;          // [E][R]           quota, staged once
  __shared__ uint32_t s_status;
  __shared__ int32_t s_carry;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The next kernel's CTAs are let in only once the previous step has finished: released earlier they sit
  // resident through that step's tail and cost it time (0.6 us per step on a decode-sized batch).
  pdl_wait();
  pdl_trigger();
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));
  const int P = nv * p.k;                     // live pairs
  const int total_pairs = p.T * p.k;

  // rows are scattered into after pass 1; every CTA pre-fills its share
#pragma unroll 1
  for (int row = cta * kDispThreads + tid; row < p.M_cap; row += NC * kDispThreads) p.row_pair[row] = -1;
#pragma unroll 1
  for (int q = P + cta * kDispThreads + tid; q < total_pairs; q += NC * kDispThreads) p.pair_row[q] = -1;
  int id_bits = 0;
  while ((1 << id_bits) < E) ++id_bits;

  // all table reads are issued up front, together with the first ids, so the kernel pays the
  // global-memory latency once
#pragma unroll 1
  for (int i = tid; i < E * R; i += kDispThreads) { rmap_s[i] = p.replica_map[i]; quota_s[i] = p.quota[i]; }
#pragma unroll 1
  for (int i = tid; i < kDispWarps * E; i += kDispThreads) hist[i] = 0;
#pragma unroll 1
  for (int i = tid; i < G; i += kDispThreads) { owner[i] = 0x7fffffff; m_inst[i] = 0; }
  if (tid == 0) s_status = 0;
  __syncthreads();

  // contiguous chunk of this CTA (a multiple of 1024 pairs) and range of this warp inside it
  const int per_cta = (((P + NC - 1) / NC) + kDispThreads - 1) & ~(kDispThreads - 1);
  const int c_begin = min(P, cta * per_cta), c_end = min(P, c_begin + per_cta);
  const int per_warp = per_cta / kDispWarps;
  const int w_begin = min(c_end, c_begin + warp * per_warp), w_end = min(c_end, w_begin + per_warp);
  uint32_t my_status = 0;

  // ---- pass 1: warp histograms -------------------------------------------------------------
  int kept[kKeep];                            // ids of the first kKeep steps, reused by pass 2
  // the ids of those steps are requested together, so a warp with several steps pays the latency once
#pragma unroll
  for (int i = 0; i < kKeep; ++i) {
    const int pidx = w_begin + 32 * i + lane;
    int e = -1;
    if (pidx < w_end) {
      e = __ldg(p.topk_ids + pidx);
      if (e < 0 || e >= E) { my_status |= TEMPO_STATUS_BAD_ID; e = -1; }
    }
    kept[i] = e;
  }
  {
    int step = 0;
    for (int base = w_begin; base < w_end; base += 32, ++step) {
      const int pidx = base + lane;
      int e = -1;
      if (step < kKeep) {
#pragma unroll
        for (int i = 0; i < kKeep; ++i) if (i == step) e = kept[i];
      } else if (pidx < w_end) {
        e = __ldg(p.topk_ids + pidx);
        if (e < 0 || e >= E) { my_status |= TEMPO_STATUS_BAD_ID; e = -1; }
      }
      const uint32_t same = same_expert_mask(e, id_bits);
      if (e >= 0 && lane == __ffs(same) - 1) hist[warp * E + e] += __popc(same);
      __syncwarp();
    }
  }
  // ---- which (e, r) owns each slot: the first entry in row-major order ----------------------
#pragma unroll 1
  for (int idx = tid; idx < E * R; idx += kDispThreads) {
    const int slot = rmap_s[idx];
    if (slot >= 0 && slot < G) atomicMin(&owner[slot], idx);
    else if (slot != -1 && cta == 0) my_status |= TEMPO_STATUS_BAD_TABLE;
  }
  __syncthreads();

  // ---- per expert: warp bases inside the CTA, CTA total -------------------------------------
#pragma unroll 1
  for (int e = tid; e < E; e += kDispThreads) {
    int run = 0;
    for (int w = 0; w < kDispWarps; ++w) {
      const int c = hist[w * E + e];
      hist[w * E + e] = run;
      run += c;
    }
    tot[e] = run;
  }
  cluster.sync();

  // ---- per expert: base over lower CTAs, n_e, replica boundaries ------------------------------
#pragma unroll 1
  for (int e = tid; e < E; e += kDispThreads) {
    int n_e = 0, base = 0;
    // the other CTAs' totals, four remote reads in flight at a time (one at a time costs a distributed-shared-memory
    // round trip per CTA of the cluster)
#pragma unroll 1
    for (int c0 = 0; c0 < NC; c0 += 4) {
      int v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = c0 + u < NC ? *cluster.map_shared_rank(tot + e, c0 + u) : 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (c0 + u < cta) base += v[u];
        n_e += v[u];
      }
    }
    cbase[e] = base;
    if (cta == 0) {
      p.counts[e] = n_e;
      if (p.cum_counts != nullptr) atomicAdd(&p.cum_counts[e], static_cast<uint32_t>(n_e));
    }

    unsigned long long S = 0;
    uint32_t vmask = 0, st = 0;
#pragma unroll 1
    for (int r = 0; r < R; ++r) {
      const int idx = e * R + r;
      const int slot = rmap_s[idx];
      const int x = quota_s[idx];
      if (slot == -1) { if (x != 0) st |= TEMPO_STATUS_BAD_TABLE; continue; }
      if (slot < 0 || slot >= G) continue;                       // flagged above
      if (owner[slot] != idx) { st |= TEMPO_STATUS_BAD_TABLE; continue; }
      vmask |= 1u << r;
      // a share outside [0, 2^30] is malformed and counts as zero: with at most 8 columns the running sum
      // stays below 2^34 and C * n_e below 2^64, so the boundaries below cannot wrap
      if (x < 0 || x > kMaxShare) st |= TEMPO_STATUS_BAD_TABLE; else S += static_cast<unsigned long long>(x);
    }
    if (cta == 0) my_status |= st;
    const bool uniform = (S == 0);
    if (uniform) S = __popc(vmask);
    unsigned long long C = 0;
    int prev = 0;
#pragma unroll 1
    for (int r = 0; r < R; ++r) {
      const int idx = e * R + r;
      const bool valid = (vmask >> r) & 1u;
      const int xq = quota_s[idx];
      if (valid) C += uniform ? 1ull : static_cast<unsigned long long>((xq < 0 || xq > kMaxShare) ? 0 : xq);
      int B = 0;
      if (S > 0) {
        if (C < 65536ull && S < 65536ull && n_e < 65536)
          B = static_cast<int>(static_cast<uint32_t>(C) * static_cast<uint32_t>(n_e) / static_cast<uint32_t>(S));
        else
          B = static_cast<int>(C * static_cast<unsigned long long>(n_e) / S);
      }
      bnd[idx] = B;
      if (valid) m_inst[rmap_s[idx]] = B - prev;
      prev = B;
    }
  }
  __syncthreads();

  // ---- padded offsets: exclusive scan of 128*ceil(m/128) in ascending slot id (warp 0) -------
  // (masked layout: instance i simply starts at row i * max_m)
  if (p.max_m > 0) {
#pragma unroll 1
    for (int i = tid; i <= G; i += kDispThreads) off[i] = i * p.max_m;
#pragma unroll 1
    for (int i = tid; i < G; i += kDispThreads)
      if (m_inst[i] > p.max_m && cta == 0) my_status |= TEMPO_STATUS_CAPACITY;
  } else if (warp == 0) {
    if (lane == 0) s_carry = 0;
    __syncwarp();
#pragma unroll 1
    for (int base = 0; base < G; base += 32) {
      const int i = base + lane;
      const int padded = i < G ? ((m_inst[i] + kTileM - 1) / kTileM) * kTileM : 0;
      int incl = padded;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const int carry = s_carry;
      if (i < G) off[i] = carry + incl - padded;
      __syncwarp();
      if (lane == 31) s_carry = carry + incl;
      __syncwarp();
    }
    if (lane == 0) off[G] = s_carry;
  }
  __syncthreads();

  const int M_pad_full = off[G];
  const int m_pad = min(M_pad_full, p.M_cap);
  if (cta == 0) {
    if (tid == 0) {
      *p.m_pad = m_pad;
      if (M_pad_full > p.M_cap) my_status |= TEMPO_STATUS_CAPACITY;
    }
#pragma unroll 1
    for (int i = tid; i <= G; i += kDispThreads) {
      p.inst_off[i] = min(off[i], p.M_cap);
      if (i < G) p.inst_count[i] = max(0, min(min(m_inst[i], p.M_cap - off[i]), p.max_m > 0 ? p.max_m : m_inst[i]));
    }
#pragma unroll 1
    for (int tau = tid; tau < p.M_cap / kTileM; tau += kDispThreads) {
      const int row = tau * kTileM;
      int inst = -1;
      if (row < m_pad) {
        int lo = 0, hi = G;                                        // first i with off[i+1] > row
#pragma unroll 1
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (off[mid + 1] > row) hi = mid; else lo = mid + 1;
        }
        inst = lo;
        // masked layout: only the tiles that hold rows belong to the instance
        if (p.max_m > 0 && row - off[lo] >= ((min(m_inst[lo], p.max_m) + kTileM - 1) / kTileM) * kTileM) inst = -1;
      }
      p.tile_inst[tau] = inst;
    }
  }
  // Nobody reads a neighbour's totals any more (a CTA must not run ahead and exit while they are being read).
  // This barrier orders no memory - the pre-fill of row_pair was ordered before the scatters below by the
  // cluster barrier after pass 1 - so it is taken without the release/acquire fences of cluster.sync().
  asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");

  // ---- pass 2: stable ranks -> replica -> row -------------------------------------------------
  int step = 0;
  for (int base = w_begin; base < w_end; base += 32, ++step) {
    const int pidx = base + lane;
    int e = -1;
    if (step < kKeep) {
#pragma unroll
      for (int i = 0; i < kKeep; ++i) if (i == step) e = kept[i];
    } else if (pidx < w_end) {
      e = __ldg(p.topk_ids + pidx);
      if (e < 0 || e >= E) e = -1;
    }
    const uint32_t same = same_expert_mask(e, id_bits);
    int j = 0;
    if (e >= 0) j = cbase[e] + hist[warp * E + e] + __popc(same & ((1u << lane) - 1u));
    __syncwarp();
    if (e >= 0 && lane == __ffs(same) - 1) hist[warp * E + e] += __popc(same);
    __syncwarp();
    if (pidx < w_end) {
      int row = -1;
      if (e >= 0) {
        int prev = 0;
        for (int r = 0; r < R; ++r) {
          const int B = bnd[e * R + r];
          if (j < B) {                                           // B only grows on valid columns
            const int cand = off[rmap_s[e * R + r]] + (j - prev);
            if (cand < p.M_cap && (p.max_m == 0 || j - prev < p.max_m)) row = cand;
            break;
          }
          prev = B;
        }
      }
      p.pair_row[pidx] = row;
      if (row >= 0) p.row_pair[row] = pidx;
    }
  }

  if (my_status) atomicOr(&s_status, my_status);
  __syncthreads();
  if (tid == 0 && s_status) atomicOr(p.status, s_status);
}

size_t dispatch_smem_bytes(int E, int R, int G) {
  return sizeof(int32_t) * (static_cast<size_t>(kDispWarps + 2) * E + 3 * static_cast<size_t>(E) * R +
                            3 * static_cast<size_t>(G) + 1);
}

cudaError_t launch_count_dispatch(const DispatchParams& p, cudaStream_t stream) {
  const size_t smem = dispatch_smem_bytes(p.E, p.R_max, p.G_max);
  return launch_dispatch_cluster(count_dispatch_kernel, p, static_cast<long long>(p.T) * p.k, smem, stream);
}

}  // namespace tempo
