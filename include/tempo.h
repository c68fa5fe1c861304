/*
 * tempo.h - C ABI of the B200 (sm_100a) per-rank MoE expert block.
 *
 * One GPU plays one expert-parallel rank.  The block is the data-parallel hot path whose
 * per-rank time the paper's dispatcher balances (Eq. 1: t_g = max(a + b*G_g, c + beta*N_g)):
 *
 *   tempo_count_dispatch     counts + quota dispatch + padded grouped layout   (Section 4.4, Eq. 2, Eq. 3)
 *   tempo_permute_pad        gather rows into the layout, fp8-quantise them    (Appendix B "scatter/gather, quantization")
 *   tempo_grouped_ffn        fp8 grouped gate/up GEMM + SwiGLU + down GEMM     (Section 2.1 "gate/up, activation, down")
 *   tempo_unpermute_combine  weighted sum over each token's k slots            (Section 2.1 "combine")
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless marked [host].  The caller owns every buffer;
 *     the library allocates nothing and keeps no state between calls that a caller could observe
 *     (two host-side caches only: the address of a driver routine, and which devices already had
 *     a kernel's shared-memory limit raised; both are safe to fill from several threads).  The
 *     one exception is tempo_grouped_ffn_static, which owns a device array: see there.
 *   - `stream` is a cudaStream_t passed as void*.  Every hot-path call only enqueues kernels:
 *     no host synchronisation, no host read of device data, no allocation, so the calls can be
 *     captured in a CUDA graph (the deployment the paper describes, Section 2.1 / 4.4).
 *     Data-dependent sizes (n_valid, m_pad, the tile list) live in device memory.
 *   - Return value: TEMPO_OK, or a negative TEMPO_ERR_* for a problem visible on the host
 *     (nothing was launched).  Data-dependent problems are OR-ed into the device word
 *     `status` (TEMPO_STATUS_* bits); the library never clears it.  Kernels never trap, never
 *     write out of bounds and never wait without a bound.
 *   - Notation: T token rows, n_valid <= T live rows (rows beyond are CUDA-graph padding and
 *     are neither counted nor dispatched, Section 4.4), k = top-k, E global logical experts,
 *     G_max instance slots on this rank (an instance = one physical copy of one expert = the
 *     paper's "(expert, replica) pair"), R_max replica columns per expert, d model dim,
 *     f FFN dim, pair index p = t*k + s.
 *
 * Layouts defined by the library
 *   - Padded grouped layout: instance slot i owns rows [inst_off[i], inst_off[i+1]), a
 *     multiple of 128 rows (Eq. 3: T = sum ceil(n/128) M-tiles); live rows first in ascending
 *     pair index ("stable by token index"), then zero rows.  Instances in ascending slot id.
 *   - fp8 is e4m3 ("fn": bias 7, max 448, no inf).  Scales are powers of two.
 *   - Activation scale bytes ("SF"): UE8M0 (byte b means 2^(b-127)), one per row per 128
 *     columns, stored in 512-byte atoms that cover 128 rows x 4 column blocks:
 *         sf_index(row, kb, K) = ((row/128) * J + kb/4) * 512 + (row%32)*16 + ((row%128)/32)*4 + kb%4,
 *         J = ceil((K/128)/4),  buffer size = tempo_sf_bytes(M_cap, K).
 *     This is the order the tensor core's scale-factor copy consumes directly.
 */
#ifndef TEMPO_H_
#define TEMPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t T, k, E;       /* token rows allocated, top-k (<= 32), global logical experts (<= 1024) */
  int32_t G_max, R_max;  /* instance slots on this rank (<= 1024), replica columns per expert (<= 8) */
  int32_t d, f;          /* model dim, FFN dim; both multiples of 128                               */
  int32_t M_cap;         /* row capacity of the padded buffers, multiple of 128                     */
} tempo_shape;

enum {
  TEMPO_OK = 0,
  TEMPO_ERR_NULL = -1,        /* a required pointer is NULL                      */
  TEMPO_ERR_SHAPE = -2,       /* a size is not positive or not a multiple of 128 */
  TEMPO_ERR_UNSUPPORTED = -3, /* a size exceeds a documented limit               */
  TEMPO_ERR_CUDA = -4         /* a CUDA call (launch, tensor-map encode) failed  */
};

enum {
  TEMPO_STATUS_BAD_ID = 1,     /* a live pair names an expert outside [0,E): pair ignored            */
  TEMPO_STATUS_BAD_TABLE = 2,  /* negative share, share on a -1 column, slot outside [0,G_max) or
                                  claimed twice: the entry counts as absent / zero                   */
  TEMPO_STATUS_CAPACITY = 4,   /* padded rows exceed M_cap: rows that do not fit are dropped         */
  TEMPO_STATUS_TIMEOUT = 8,    /* a bounded device wait expired; the outputs of that call are invalid */
  TEMPO_STATUS_BAD_SCALE = 16  /* tempo_pack_weights met a weight scale that is not a power of two   */
};

int tempo_version(void);

const char* tempo_status_string(int code); /* [host] text for a TEMPO_ERR_* code */

/* [host] Safe row capacity: round128(T*k) + 128*G_max (each instance pads by < 128 rows). */
int tempo_m_cap_bound(const tempo_shape* shape /*[host]*/, int32_t* m_cap /*[host]*/);

/* [host] Bytes of a scale-byte buffer for an operand of `rows` x `cols` (see sf_index above). */
int tempo_sf_bytes(int32_t rows, int32_t cols, size_t* bytes /*[host]*/);

/*
 * [host] Bytes of the scratch buffer of tempo_grouped_ffn: two int32 counters per 128-row tile of
 * the padded layout (8 * M_cap / 128, rounded up to 256).  The caller allocates it and ZEROES it
 * once; every call that completes leaves it zero again.  After a call that reported
 * TEMPO_STATUS_TIMEOUT zero it again.  Calls that may overlap on the GPU need a buffer each.
 */
int tempo_workspace_bytes(const tempo_shape* shape /*[host]*/, size_t* bytes /*[host]*/);

/* [host] Bytes of the packed weight blob for G_max instances of shape (d, f). */
int tempo_packed_weight_bytes(const tempo_shape* shape /*[host]*/, size_t* bytes /*[host]*/);

/*
 * One-time, off the hot path: re-lay the weights of all G_max instance slots for the GEMM
 * kernels.  Every replica slot owns its own copy of its expert's weights: touching one more
 * instance costs one more weight stream, which is the activation floor b of Eq. 1.
 *   w13_q  u8  [G_max, 2f, d]  e4m3 codes, rows [0,f) gate projection, [f,2f) up projection
 *   w13_s  f32 [G_max, 2f/128, d/128]  one power-of-two scale per 128x128 block
 *   w2_q   u8  [G_max, d, f]   down projection;  w2_s f32 [G_max, d/128, f/128]
 *   packed u8  [tempo_packed_weight_bytes]  (256-byte aligned): gate/up rows interleaved per
 *          128-column block of H so one tile holds both halves of SwiGLU, plus UE8M0 scale atoms.
 * A scale that is not a positive power of two sets TEMPO_STATUS_BAD_SCALE in *status.
 */
int tempo_pack_weights(const tempo_shape* shape, const void* w13_q, const float* w13_s, const void* w2_q,
                       const float* w2_s, void* packed, uint32_t* status, void* stream);

/*
 * Step 1 (Section 4.4: dispatch fused with count collection; Eq. 2: shares x_{e,r} >= 0 supported on
 * R(e) with sum_r x_{e,r} = n_e; Eq. 3: 128-row tiles).  One kernel.
 *   in   topk_ids    i32 [T, k]       router output
 *        n_valid     i32 [1] or NULL  live rows (NULL: T); clamped to [0, T]
 *        replica_map i32 [E, R_max]   instance slot holding replica column r of expert e, -1 = none
 *        quota       i32 [E, R_max]   share x_{e,r} of expert e's pairs for that column
 *   out  counts      i32 [E]          n_e over live rows, all E experts (local or not)
 *        cum_counts  u32 [E] or NULL  += counts, wraps mod 2^32 (persistent, never zeroed)
 *        inst_count  i32 [G_max]      live rows of each instance
 *        inst_off    i32 [G_max+1]    first row of each instance; inst_off[G_max] = m_pad
 *        pair_row    i32 [T*k]        row of pair p, or -1 (dead row, remote expert, bad id, dropped)
 *        row_pair    i32 [M_cap]      pair held by each row, -1 for padding rows and rows >= m_pad
 *        tile_inst   i32 [M_cap/128]  instance of each 128-row tile, -1 beyond m_pad/128
 *        m_pad       i32 [1]          padded rows in use = sum_i 128*ceil(inst_count[i]/128), <= M_cap
 * Replica choice: the pairs of expert e are ranked by ascending p; with q_r = max(quota,0) on
 * columns that hold the expert, S = sum q_r (all q_r = 1 if S == 0: uniform fallback), column r
 * takes ranks [floor(C_{r-1} n_e / S), floor(C_r n_e / S)), C the running sum of q.  When
 * S == n_e every column receives exactly its share.  A pair can never go to a column whose
 * slot is -1, and nothing divides by zero.  A share above 2^30 is a malformed entry like a negative
 * one (counts as zero, TEMPO_STATUS_BAD_TABLE), so the 64-bit products above cannot wrap.
 */
int tempo_count_dispatch(const tempo_shape* shape, const int32_t* topk_ids, const int32_t* n_valid,
                         const int32_t* replica_map, const int32_t* quota, uint32_t* cum_counts,
                         int32_t* counts, int32_t* inst_count, int32_t* inst_off, int32_t* pair_row,
                         int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad, uint32_t* status, void* stream);

/*
 * Step 1, sampled variant: the in-graph kernel as Section 4.4 describes it.  Same outputs and layout as
 * tempo_count_dispatch, but the replica of each pair is drawn from its expert's row of a FLOAT share table:
 *   table  f32 [E, R_max]  non-negative shares; only columns whose replica_map entry holds the expert
 *          count; the row is renormalised at use; a row that sums to zero (or whose shares are all
 *          invalid) falls back to uniform over the holders; negative / NaN / infinite shares, and shares
 *          on a -1 column, count as zero and set TEMPO_STATUS_BAD_TABLE.  A torn or stale row therefore
 *          costs a batch a stale or uniform split, never a wrong replica.
 *   seed, layer  the draw for pair p is word 0 of Philox-4x32-10 with key (seed low, seed high) and counter
 *          (p, 0, layer, 0): u = (word >> 8) * 2^-24; column = first holder r with u*S < C_r, S and the running
 *          sums C_r accumulated in fp32 in column order (last holder if rounding leaves none).  The result is a
 *          pure function of the arguments: replaying a graph with the same seed and layer repeats the dispatch;
 *          advance `layer` (or the seed) per call for fresh draws.
 * Rows of an instance are in ascending pair index.
 */
int tempo_count_dispatch_sampled(const tempo_shape* shape, const int32_t* topk_ids, const int32_t* n_valid,
                                 const int32_t* replica_map, const float* table, uint64_t seed, uint32_t layer,
                                 uint32_t* cum_counts, int32_t* counts, int32_t* inst_count, int32_t* inst_off,
                                 int32_t* pair_row, int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad,
                                 uint32_t* status, void* stream);

/*
 * Step 2.  a_q[row,:] = e4m3(x[row_pair[row]/k, :] / 2^eps) per 128-column block, eps the smallest
 * integer with max|block| <= 448 * 2^eps (0 for an all-zero block), round-to-nearest-even,
 * saturating; padding rows are zero codes with scale 1.  Rows >= m_pad are not written.
 *   in   x bf16 [T, d], row_pair, m_pad        out  a_q u8 [M_cap, d], a_sf u8 [tempo_sf_bytes(M_cap, d)]
 *   pair_row (optional, may be NULL): step 1's pair -> row map.  Without it the kernel walks the ROWS of
 *   the layout and gathers.  With it the kernel may walk the TOKENS instead, quantising each row of x once
 *   and writing it to the rows of all its local pairs: for batches small enough that every (token, 512
 *   columns) item gets a warp of its own or up to six items per warp (decode-sized), in one wave with no
 *   loop; and for batches whose x no longer stays in L2 between a token's gathers (T*d*2 > 48 MB), with a
 *   grid-stride loop, so x is read from HBM once however many local pairs a token has.  In between
 *   it walks the rows.  Same output bit for bit whichever walk runs.  pair_row and row_pair must come from
 *   the same step-1 call.
 */
int tempo_permute_pad(const tempo_shape* shape, const void* x_bf16, const int32_t* row_pair,
                      const int32_t* pair_row, const int32_t* m_pad, void* a_q, uint8_t* a_sf,
                      uint32_t* status, void* stream);

/*
 * Step 3a: per instance GU = A * W13^T (fp8 x fp8 -> fp32 on the tensor cores, block scales applied
 * by the MMA), H = silu(gate) * up, then H is re-quantised like step 2 along f.
 *   in   a_q, a_sf, packed, inst_off, m_pad    out  h_q u8 [M_cap, f], h_sf u8 [tempo_sf_bytes(M_cap, f)]
 * Step 3b: Y = Hq * W2^T, stored as bf16.       out  y bf16 [M_cap, d]
 * tempo_grouped_ffn runs 3a and 3b in ONE kernel: the down tiles of a 128-row tile start as soon as
 * its H blocks are complete (tracked in `workspace`, see tempo_workspace_bytes), so the weight
 * stream never pauses between the two GEMMs.  The kernel's CTAs wait for each other's H blocks
 * (bounded, one per SM): launch it on a GPU it does not have to share with another long-running
 * kernel, or the wait may time out (TEMPO_STATUS_TIMEOUT).  Rows >= m_pad are not written.
 * Every device-side wait of the kernel gives up after 50 ms (the longest wait of a healthy launch is a
 * few milliseconds on the largest shapes); tempo_grouped_ffn_bounded is the same call with the bound
 * as an argument (nanoseconds, > 0), for a GPU shared through MPS or time slicing, where a CTA can be
 * kept off its SM for longer: give it a few times the longest kernel of the co-tenant.
 */
int tempo_ffn_gate_up(const tempo_shape* shape, const void* a_q, const uint8_t* a_sf, const void* packed,
                      const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf,
                      uint32_t* status, void* stream);
int tempo_ffn_down(const tempo_shape* shape, const void* h_q, const uint8_t* h_sf, const void* packed,
                   const int32_t* inst_off, const int32_t* m_pad, void* y_bf16, uint32_t* status, void* stream);
int tempo_grouped_ffn(const tempo_shape* shape, const void* a_q, const uint8_t* a_sf, const void* packed,
                      const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                      uint32_t* status, void* workspace, void* stream);

int tempo_grouped_ffn_bounded(const tempo_shape* shape, const void* a_q, const uint8_t* a_sf, const void* packed,
                              const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                              uint32_t* status, void* workspace, uint64_t wait_limit_ns, void* stream);

/*
 * Steps 2 and 3 with the gather fused into the GEMM (Appendix B counts "scatter/gather, quantization" among
 * the un-fused per-token kernels that multiply the per-token slope at pipeline scope; this pair removes the
 * permuted copy).  Same results as tempo_permute_pad + tempo_grouped_ffn, bit for bit.
 *   tempo_quantize_tokens     x_q[t,:] = e4m3(x[t,:] / 2^eps) per 128-column block for every live token
 *                             (t < n_valid), the rule of step 2; x_sf[t*S + kb] = eps + 127 (UE8M0), S =
 *                             4*ceil((d/128)/4) bytes per token (tempo_token_sf_bytes gives T*S).  It reads
 *                             nothing step 1 writes: enqueued right after tempo_count_dispatch on the same
 *                             stream it runs beside it, and still finishes only after it.
 *        in  x bf16 [T, d], n_valid (or NULL)      out  x_q u8 [T, d], x_sf u8 [T*S]
 *   tempo_grouped_ffn_gather  tempo_grouped_ffn whose gate/up GEMM fetches row r of its operand from
 *                             x_q[row_pair[r] / k, :] (rows with row_pair[r] < 0 are zero rows) while it fills
 *                             its shared-memory stages: a_q / a_sf are never materialised.  Same `workspace`,
 *                             waits and status bits as tempo_grouped_ffn.
 */
int tempo_token_sf_bytes(const tempo_shape* shape /*[host]*/, size_t* bytes /*[host]*/);
int tempo_quantize_tokens(const tempo_shape* shape, const void* x_bf16, const int32_t* n_valid, void* x_q,
                          uint8_t* x_sf, uint32_t* status, void* stream);
int tempo_grouped_ffn_gather(const tempo_shape* shape, const void* x_q, const uint8_t* x_sf, const int32_t* row_pair,
                             const void* packed, const int32_t* inst_off, const int32_t* m_pad, void* h_q,
                             uint8_t* h_sf, void* y_bf16, uint32_t* status, void* workspace, void* stream);

/*
 * tempo_grouped_ffn without a caller-provided scratch buffer.  (The paper has no counterpart: this
 * exists for the integration, not for the method.)  Some callers cannot allocate device memory at
 * the point where they need the FFN: code that runs after the serving process has frozen its
 * memory pool, a plug-in that is only handed the tensors of the layer, or a loop that must not
 * risk the implicit device synchronisation cudaMalloc can cause.  For them the counters live in
 * a 128 KB array built into the library image (one copy on every GPU that loads the library, held
 * until the process exits).
 *   - Same arguments, results and status bits as tempo_grouped_ffn, minus `workspace`.
 *   - Limit: M_cap <= 2,097,152 rows (16384 tiles of 128).  A larger M_cap returns
 *     TEMPO_ERR_UNSUPPORTED and launches nothing.
 *   - Allocates nothing, ever.  The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and caches it on the host (atomically: two
 *     threads racing on a device's first call both look the address up and store the same value);
 *     make that first call outside any stream capture.  Every call enqueues a small cudaMemsetAsync of the counters before the kernel.
 *   - All calls on a GPU share the one array: two calls that can overlap on the GPU (different
 *     streams) race on it and give wrong results.  Serialise them, or use tempo_grouped_ffn with a
 *     buffer per stream.
 */
int tempo_grouped_ffn_static(const tempo_shape* shape, const void* a_q, const uint8_t* a_sf, const void* packed,
                             const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                             uint32_t* status, void* stream);

/*
 * Step 4.  out[t,:] = sum_{s<k, pair_row[t*k+s] >= 0} topk_w[t,s] * y[pair_row[t*k+s], :], slots in
 * ascending order, fp32 accumulation, bf16 store.  Rows t >= n_valid and rows with no local pair are zero.
 *   in   y bf16 [M_cap, d], pair_row, topk_w f32 [T, k], n_valid (or NULL)     out  out bf16 [T, d]
 */
int tempo_unpermute_combine(const tempo_shape* shape, const void* y_bf16, const int32_t* pair_row,
                            const float* topk_w, const int32_t* n_valid, void* out_bf16, uint32_t* status,
                            void* stream);

/*
 * Masked layout (the layout of the masked grouped GEMM the paper calibrates for decode, Section 2.1 and
 * Appendix B): instance i owns the FIXED row range [i*max_m, (i+1)*max_m) of every padded buffer and uses
 * its first inst_count[i] rows; nothing moves when the counts change from step to step.  max_m is a
 * multiple of 128 with G_max*max_m <= M_cap (TEMPO_ERR_SHAPE otherwise).
 *   tempo_count_dispatch_masked  as tempo_count_dispatch with inst_off[i] = i*max_m, m_pad = G_max*max_m,
 *        tile_inst[tile] = i only for the ceil(inst_count[i]/128) tiles of instance i that hold rows (-1
 *        elsewhere); pairs beyond max_m rows of an instance are dropped (pair_row = -1, TEMPO_STATUS_CAPACITY).
 *   tempo_permute_pad_masked     step 2 for that layout: writes the rows of the tiles in use (rows with a pair,
 *        zero rows up to the next tile boundary) and leaves unused tiles alone.
 *   tempo_grouped_ffn_masked     step 3 (one kernel, as tempo_grouped_ffn) on the tiles in use only.
 * Step 4 is tempo_unpermute_combine.  Results per row are those of the grouped layout bit for bit.
 */
int tempo_count_dispatch_masked(const tempo_shape* shape, int32_t max_m, const int32_t* topk_ids,
                                const int32_t* n_valid, const int32_t* replica_map, const int32_t* quota,
                                uint32_t* cum_counts, int32_t* counts, int32_t* inst_count, int32_t* inst_off,
                                int32_t* pair_row, int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad,
                                uint32_t* status, void* stream);
int tempo_permute_pad_masked(const tempo_shape* shape, const void* x_bf16, const int32_t* row_pair,
                             const int32_t* pair_row, const int32_t* tile_inst, const int32_t* m_pad, void* a_q,
                             uint8_t* a_sf, uint32_t* status, void* stream);
int tempo_grouped_ffn_masked(const tempo_shape* shape, int32_t max_m, const void* a_q, const uint8_t* a_sf,
                             const void* packed, const int32_t* inst_count, void* h_q, uint8_t* h_sf, void* y_bf16,
                             uint32_t* status, void* workspace, void* stream);

/*
 * bf16 variant of steps 2 and 3 (the paper calibrates a bf16 grouped GEMM beside the fp8 one and finds
 * the same two-regime shape with a later inflection: Section 2.1, Table "Fitted cost parameters").
 * No quantiser: the gathered rows stay bf16, both GEMMs multiply bf16 values with fp32 accumulation
 * on the tensor cores, H = silu(gate) * up is rounded to bf16 (nearest even) before the down GEMM,
 * Y is stored as bf16.  Steps 1 and 4 are the calls above.
 *   tempo_packed_weight_bytes_bf16 [host]  bytes of the packed bf16 blob (6*d*f per instance, padded)
 *   tempo_pack_weights_bf16   one-time re-layout of w13 bf16 [G_max, 2f, d] (rows [0,f) gate, [f,2f) up)
 *                             and w2 bf16 [G_max, d, f] into tiles of 256 rows x 64 values
 *   tempo_permute_pad_bf16    a[row,:] = x[row_pair[row]/k, :], zero for rows without a pair; rows >= m_pad
 *                             are not written.          out  a bf16 [M_cap, d]
 *   tempo_grouped_ffn_bf16    both GEMMs in one kernel, as tempo_grouped_ffn (same `workspace`, same
 *                             bounded waits and TEMPO_STATUS_TIMEOUT).   out  h bf16 [M_cap, f], y bf16 [M_cap, d]
 */
int tempo_packed_weight_bytes_bf16(const tempo_shape* shape /*[host]*/, size_t* bytes /*[host]*/);
int tempo_pack_weights_bf16(const tempo_shape* shape, const void* w13_bf16, const void* w2_bf16, void* packed,
                            void* stream);
int tempo_permute_pad_bf16(const tempo_shape* shape, const void* x_bf16, const int32_t* row_pair,
                           const int32_t* m_pad, void* a_bf16, uint32_t* status, void* stream);
int tempo_grouped_ffn_bf16(const tempo_shape* shape, const void* a_bf16, const void* packed,
                           const int32_t* inst_off, const int32_t* m_pad, void* h_bf16, void* y_bf16,
                           uint32_t* status, void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TEMPO_H_ */
