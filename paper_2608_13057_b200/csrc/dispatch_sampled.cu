// Step 1, sampled variant: the in-graph kernel as the paper deploys it (Section 4.4).  The replica of
// every (token, slot) pair is DRAWN from the pair's expert row of a float share table: the row is
// renormalised at use (only columns that hold the expert count), a row that sums to zero falls back
// to uniform over the replicas holding the expert, a pair can never go to a column whose slot is -1,
// nothing divides.  Count collection into the cumulative per-expert counter is fused in, padding
// rows are masked.
//
// The draw is a counter-based generator, Philox-4x32-10 keyed by the caller's seed and indexed by
// (pair index, layer), so the result is a pure function of the inputs and a CPU oracle can
// reproduce it bit for bit: u = (word0 >> 8) * 2^-24, column = first holder r with u*S < C_r where
// S and the running sums C_r are accumulated in fp32 in column order.
//
// Layout work is the same as in the quota kernel with the instance slot as the sort key: per-warp
// histograms over slots, prefix over warps and over the CTAs of the cluster, then a second pass
// that gives every pair its row (rows of an instance in ascending pair index).  Per-expert counts are
// order-free and use shared-memory atomics.
#include <cooperative_groups.h>

#include "dispatch_common.cuh"

namespace cg = cooperative_groups;

namespace tempo {

__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

// Instance slot drawn for pair p of expert e, or -1 if the expert is not on this rank.
__device__ __forceinline__ int draw_slot(int e, int pidx, const SampledParams& p, const int32_t* rmap_s,
                                         const float* share_s, const uint32_t* vmask_s) {
  const int R = p.R_max;
  const uint32_t vmask = vmask_s[e];
  if (vmask == 0) return -1;
  float S = 0.f;
  for (int r = 0; r < R; ++r)
    if ((vmask >> r) & 1u) S = __fadd_rn(S, share_s[e * R + r]);
  const bool uniform = !(S > 0.f);
  if (uniform) S = static_cast<float>(__popc(vmask));
  const uint32_t w0 = philox4x32_10_word0(static_cast<uint32_t>(pidx), 0u, p.layer, 0u,
                                          static_cast<uint32_t>(p.seed), static_cast<uint32_t>(p.seed >> 32));
  const float u = __fmul_rn(static_cast<float>(w0 >> 8), 5.9604644775390625e-08f);   // 2^-24
  const float thr = __fmul_rn(u, S);
  float C = 0.f;
  int pick = 31 - __clz(vmask);                           // last holder, if rounding leaves thr >= C_last
  for (int r = 0; r < R; ++r) {
    if (!((vmask >> r) & 1u)) continue;
    C = __fadd_rn(C, uniform ? 1.f : share_s[e * R + r]);
    if (thr < C) { pick = r; break; }
  }
  return rmap_s[e * R + pick];
}

__global__ void __launch_bounds__(kDispThreads, 1) count_dispatch_sampled_kernel(const SampledParams p) {
  extern __shared__ int32_t smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int NC = static_cast<int>(cluster.num_blocks());
  const int cta = static_cast<int>(cluster.block_rank());
  const int E = p.E, R = p.R_max, G = p.G_max;
  int32_t* hist = smem;                                    // [kDispWarps][G]  warp histograms over slots
  int32_t* tot = hist + kDispWarps * G;                    // [G]   this CTA's rows per slot (read by the other CTAs)
  int32_t* cbase = tot + G;                                // [G]   rows of the slot in lower-ranked CTAs
  int32_t* owner = cbase + G;                              // [G]   first (e,r) entry naming the slot
  int32_t* m_inst = owner + G;                             // [G]   rows of each instance
  int32_t* off = m_inst + G;                               // [G+1] padded offsets (not clamped)
  int32_t* ecount = off + G + 1;                           // [E]   this CTA's pairs per expert (read by CTA 0)
  int32_t* rmap_s = ecount + E;                            // [E][R]
  float* share_s = reinterpret_cast<float*>(rmap_s + E * R);       // [E][R] cleaned shares
  uint32_t* vmask_s = reinterpret_cast<uint32_t*>(share_s + E * R);  // [E] columns that hold the expert
  __shared__ uint32_t s_status;
  __shared__ int32_t s_carry;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The next kernel's CTAs are let in only once the previous step has finished: released earlier they sit
  // resident through that step's tail and cost it time (0.6 us per step on a decode-sized batch).
  pdl_wait();
  pdl_trigger();
  int nv = p.T;
  if (p.n_valid != nullptr) nv = max(0, min(*p.n_valid, p.T));
  const int P = nv * p.k;
  const int total_pairs = p.T * p.k;

  for (int row = cta * kDispThreads + tid; row < p.M_cap; row += NC * kDispThreads) p.row_pair[row] = -1;
  for (int q = P + cta * kDispThreads + tid; q < total_pairs; q += NC * kDispThreads) p.pair_row[q] = -1;
  int slot_bits = 0;
  while ((1 << slot_bits) < G) ++slot_bits;

  for (int i = tid; i < E * R; i += kDispThreads) rmap_s[i] = p.replica_map[i];
  for (int i = tid; i < kDispWarps * G; i += kDispThreads) hist[i] = 0;
  for (int i = tid; i < G; i += kDispThreads) { owner[i] = 0x7fffffff; m_inst[i] = 0; }
  for (int i = tid; i < E; i += kDispThreads) ecount[i] = 0;
  if (tid == 0) s_status = 0;
  __syncthreads();
  uint32_t my_status = 0;
  for (int idx = tid; idx < E * R; idx += kDispThreads) {
    const int slot = rmap_s[idx];
    if (slot >= 0 && slot < G) atomicMin(&owner[slot], idx);
    else if (slot != -1 && cta == 0) my_status |= TEMPO_STATUS_BAD_TABLE;
  }
  __syncthreads();
  // holders and cleaned shares per expert
  for (int e = tid; e < E; e += kDispThreads) {
    uint32_t vmask = 0, st = 0;
    for (int r = 0; r < R; ++r) {
      const int idx = e * R + r;
      const int slot = rmap_s[idx];
      float x = p.table[idx];
      if (slot == -1) { if (x != 0.f || x != x) st |= TEMPO_STATUS_BAD_TABLE; share_s[idx] = 0.f; continue; }
      if (slot < 0 || slot >= G) { share_s[idx] = 0.f; continue; }
      if (owner[slot] != idx) { st |= TEMPO_STATUS_BAD_TABLE; share_s[idx] = 0.f; continue; }
      vmask |= 1u << r;
      if (!(x >= 0.f) || x > 3.402823466e38f) { st |= TEMPO_STATUS_BAD_TABLE; x = 0.f; }   // negative, NaN, inf
      share_s[idx] = x;
    }
    vmask_s[e] = vmask;
    if (cta == 0) my_status |= st;
  }
  __syncthreads();

  const int per_cta = (((P + NC - 1) / NC) + kDispThreads - 1) & ~(kDispThreads - 1);
  const int c_begin = min(P, cta * per_cta), c_end = min(P, c_begin + per_cta);
  const int per_warp = per_cta / kDispWarps;
  const int w_begin = min(c_end, c_begin + warp * per_warp), w_end = min(c_end, w_begin + per_warp);

  // ---- pass 1: draw, count experts, warp histograms over slots --------------------------------
  int kept[kKeep];
#pragma unroll
  for (int i = 0; i < kKeep; ++i) kept[i] = -1;
  {
    int step = 0;
    for (int base = w_begin; base < w_end; base += 32, ++step) {
      const int pidx = base + lane;
      int slot = -1;
      if (pidx < w_end) {
        const int e = __ldg(p.topk_ids + pidx);
        if (e < 0 || e >= E) my_status |= TEMPO_STATUS_BAD_ID;
        else {
          atomicAdd(&ecount[e], 1);
          slot = draw_slot(e, pidx, p, rmap_s, share_s, vmask_s);
        }
      }
#pragma unroll
      for (int i = 0; i < kKeep; ++i) if (i == step) kept[i] = slot;
      const uint32_t same = same_expert_mask(slot, slot_bits);
      if (slot >= 0 && lane == __ffs(same) - 1) hist[warp * G + slot] += __popc(same);
      __syncwarp();
    }
  }
  __syncthreads();
  for (int i = tid; i < G; i += kDispThreads) {
    int run = 0;
    for (int w = 0; w < kDispWarps; ++w) {
      const int c = hist[w * G + i];
      hist[w * G + i] = run;
      run += c;
    }
    tot[i] = run;
  }
  cluster.sync();

  for (int i = tid; i < G; i += kDispThreads) {
    int total = 0, base = 0;
    for (int c = 0; c < NC; ++c) {
      const int v = c == cta ? tot[i] : *cluster.map_shared_rank(tot + i, c);
      if (c < cta) base += v;
      total += v;
    }
    cbase[i] = base;
    m_inst[i] = total;
  }
  if (cta == 0) {
    for (int e = tid; e < E; e += kDispThreads) {
      int n_e = 0;
      for (int c = 0; c < NC; ++c) n_e += c == 0 ? ecount[e] : *cluster.map_shared_rank(ecount + e, c);
      p.counts[e] = n_e;
      if (p.cum_counts != nullptr) atomicAdd(&p.cum_counts[e], static_cast<uint32_t>(n_e));
    }
  }
  __syncthreads();
  if (warp == 0) padded_offsets_warp0(m_inst, off, G, lane, &s_carry);
  __syncthreads();

  const int M_pad_full = off[G];
  const int m_pad = min(M_pad_full, p.M_cap);
  if (cta == 0) {
    if (tid == 0) {
      *p.m_pad = m_pad;
      if (M_pad_full > p.M_cap) my_status |= TEMPO_STATUS_CAPACITY;
    }
    for (int i = tid; i <= G; i += kDispThreads) {
      p.inst_off[i] = min(off[i], p.M_cap);
      if (i < G) p.inst_count[i] = max(0, min(m_inst[i], p.M_cap - off[i]));
    }
    for (int tau = tid; tau < p.M_cap / kTileM; tau += kDispThreads) {
      const int row = tau * kTileM;
      p.tile_inst[tau] = row < m_pad ? instance_of_row(off, G, row) : -1;
    }
  }
  cluster.sync();   // row_pair is pre-filled everywhere; nobody reads a neighbour's shared memory any more

  // ---- pass 2: rows ----------------------------------------------------------------------------
  int step = 0;
  for (int base = w_begin; base < w_end; base += 32, ++step) {
    const int pidx = base + lane;
    int slot = -1;
    if (step < kKeep) {
#pragma unroll
      for (int i = 0; i < kKeep; ++i) if (i == step) slot = kept[i];
    } else if (pidx < w_end) {
      const int e = __ldg(p.topk_ids + pidx);
      if (e >= 0 && e < E) slot = draw_slot(e, pidx, p, rmap_s, share_s, vmask_s);
    }
    const uint32_t same = same_expert_mask(slot, slot_bits);
    int j = 0;
    if (slot >= 0) j = cbase[slot] + hist[warp * G + slot] + __popc(same & ((1u << lane) - 1u));
    __syncwarp();
    if (slot >= 0 && lane == __ffs(same) - 1) hist[warp * G + slot] += __popc(same);
    __syncwarp();
    if (pidx < w_end) {
      int row = -1;
      if (slot >= 0) {
        const int cand = off[slot] + j;
        if (cand < p.M_cap) row = cand;
      }
      p.pair_row[pidx] = row;
      if (row >= 0) p.row_pair[row] = pidx;
    }
  }

  if (my_status) atomicOr(&s_status, my_status);
  __syncthreads();
  if (tid == 0 && s_status) atomicOr(p.status, s_status);
}

size_t dispatch_sampled_smem_bytes(int E, int R, int G) {
  return sizeof(int32_t) * (static_cast<size_t>(kDispWarps + 5) * G + 1 + 2 * static_cast<size_t>(E) +
                            2 * static_cast<size_t>(E) * R);
}

cudaError_t launch_count_dispatch_sampled(const SampledParams& p, cudaStream_t stream) {
  const size_t smem = dispatch_sampled_smem_bytes(p.E, p.R_max, p.G_max);
  return launch_dispatch_cluster(count_dispatch_sampled_kernel, p, static_cast<long long>(p.T) * p.k, smem, stream);
}

}  // namespace tempo
