// Parameter blocks and launchers shared between the kernel files and the C-ABI host code.
#pragma once

#include <cuda.h>

#include "tempo_common.cuh"

namespace tempo {

struct DispatchParams {
  int T, k, E, G_max, R_max, M_cap;
  const int32_t* topk_ids;
  const int32_t* n_valid;
  const int32_t* replica_map;
  const int32_t* quota;
  uint32_t* cum_counts;
  int32_t* counts;
  int32_t* inst_count;
  int32_t* inst_off;
  int32_t* pair_row;
  int32_t* row_pair;
  int32_t* tile_inst;
  int32_t* m_pad;
  uint32_t* status;
  int max_m;   // 0: instances follow each other in whole tiles; M > 0: masked layout, instance i owns rows [i*M, (i+1)*M)
};
size_t dispatch_smem_bytes(int E, int R, int G);

struct SampledParams {
  int T, k, E, G_max, R_max, M_cap;
  const int32_t* topk_ids;
  const int32_t* n_valid;
  const int32_t* replica_map;
  const float* table;
  unsigned long long seed;
  uint32_t layer;
  uint32_t* cum_counts;
  int32_t* counts;
  int32_t* inst_count;
  int32_t* inst_off;
  int32_t* pair_row;
  int32_t* row_pair;
  int32_t* tile_inst;
  int32_t* m_pad;
  uint32_t* status;
};
size_t dispatch_sampled_smem_bytes(int E, int R, int G);
cudaError_t launch_count_dispatch_sampled(const SampledParams& p, cudaStream_t stream);
cudaError_t launch_count_dispatch(const DispatchParams& p, cudaStream_t stream);

struct PermuteParams {
  int k, d, M_cap;
  const __nv_bfloat16* x;
  const int32_t* row_pair;
  int T;                      // token rows (token-major form only)
  const int32_t* pair_row;    // NULL: row-major form (gather per row); else token-major form (quantise once per token)
  const int32_t* tile_inst;   // masked layout only (else NULL): tiles with -1 hold no rows and are left alone
  const int32_t* m_pad;
  uint8_t* a_q;
  uint8_t* a_sf;
};
cudaError_t launch_permute_pad(const PermuteParams& p, int num_sms, cudaStream_t stream);
cudaError_t launch_permute_pad_bf16(const PermuteParams& p, __nv_bfloat16* a, int num_sms, cudaStream_t stream);

struct QuantizeParams {
  int T, d;
  int sf_stride;              // bytes per token of x_sf: 4 * ceil((d / 128) / 4)
  const __nv_bfloat16* x;
  const int32_t* n_valid;
  uint8_t* x_q;
  uint8_t* x_sf;
};
cudaError_t launch_quantize_tokens(const QuantizeParams& p, int num_sms, cudaStream_t stream);

struct CombineParams {
  int T, k, d;
  const __nv_bfloat16* y;
  const int32_t* pair_row;
  const float* topk_w;
  const int32_t* n_valid;
  __nv_bfloat16* out;
};
cudaError_t launch_combine(const CombineParams& p, cudaStream_t stream);

struct PackLayout {
  size_t off_w13, off_w2, off_sf13, off_sf2, total;
  int J1, J2, NT1, NT2;
};
PackLayout pack_layout(int G, int d, int f);
PackLayout pack_layout_bf16(int G, int d, int f);   // off_w13, off_w2, NT1, NT2, total only
cudaError_t launch_pack_bf16(int G, int d, int f, const __nv_bfloat16* w13, const __nv_bfloat16* w2, uint8_t* packed,
                             cudaStream_t stream);
cudaError_t launch_pack(int G, int d, int f, const uint8_t* w13_q, const float* w13_s, const uint8_t* w2_q,
                        const float* w2_s, uint8_t* packed, uint32_t* status, cudaStream_t stream);

// One of the two GEMMs of the FFN as the fused kernel sees it.
struct GemmSide {
  int Kb;        // K / 128
  int JK;        // scale atoms along K = ceil(Kb / 4)
  int NT;        // 256-column tiles per instance
  const uint8_t* wt;     // packed B tiles, 32 KB each, [inst][nt][kb]
  const uint8_t* sfa;    // scale atoms of the A operand
  const uint8_t* sfb;    // scale atoms of the packed weights
};

struct FfnParams {
  GemmSide side[2];      // 0: gate/up (A = a_q), 1: down (A = h_q)
  int run_mask;          // bit 0: run the gate/up tiles, bit 1: run the down tiles
  int G_max, M_cap;
  int d, f;
  int J_h;               // scale atoms along f of the H buffer
  const int32_t* inst_off;
  const int32_t* m_pad;
  // masked layout (stride_tiles > 0): instance i owns the M-tiles [i*stride_tiles, (i+1)*stride_tiles) and
  // uses the first ceil(inst_count[i]/128) of them; inst_off and m_pad are not read
  int stride_tiles;
  const int32_t* inst_count;
  uint8_t* h_q;
  uint8_t* h_sf;
  __nv_bfloat16* y;
  // gather form (ffn_kernel<false, true>): the gate/up operand rows are fetched from the per-token buffers
  const uint8_t* x_q;        // e4m3 codes [T, d]
  const uint8_t* x_sf;       // scale bytes [T, x_sf_stride]
  const int32_t* row_pair;   // row -> pair (token = pair / k), -1: zero row
  int x_sf_stride, k, T;
  int32_t* ready;        // workspace: per M-tile, epilogue warps of finished gate/up tiles
  int32_t* done;         // workspace: per M-tile, down tiles that have seen `ready` complete
  uint32_t* status;
  unsigned long long wait_ns;   // bound of every device-side wait of the kernel, in nanoseconds
};
size_t ffn_workspace_bytes(int M_cap);
// The bf16 variant: Kb counts 64-value K-blocks, the scale pointers and J_h are unused, h_q holds bf16.
cudaError_t launch_ffn_bf16(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmY,
                            const FfnParams& p, int num_sms, cudaStream_t stream);
cudaError_t launch_ffn(const CUtensorMap& tmA1, const CUtensorMap& tmA2, const CUtensorMap& tmY,
                       const FfnParams& p, int num_sms, cudaStream_t stream);
cudaError_t launch_ffn_gather(const CUtensorMap& tmA2, const CUtensorMap& tmY, const FfnParams& p, int num_sms,
                              cudaStream_t stream);


}  // namespace tempo
