// Host side of the C ABI: argument checks, tensor-map encoding, kernel launches.
// Nothing here synchronises, allocates or reads device memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include "tempo_kernels.cuh"

namespace tempo {

// ---- helpers ------------------------------------------------------------------------------------
constexpr int kMaxE = 1024, kMaxG = 1024, kMaxR = 8, kMaxTopK = 32;

static int check_shape(const tempo_shape* s) {
  if (s == nullptr) return TEMPO_ERR_NULL;
  if (s->T <= 0 || s->k <= 0 || s->E <= 0 || s->G_max <= 0 || s->R_max <= 0 || s->d <= 0 || s->f <= 0 || s->M_cap <= 0)
    return TEMPO_ERR_SHAPE;
  if (s->d % 128 || s->f % 128 || s->M_cap % 128) return TEMPO_ERR_SHAPE;
  if (s->E > kMaxE || s->G_max > kMaxG || s->R_max > kMaxR || s->k > kMaxTopK) return TEMPO_ERR_UNSUPPORTED;
  if (static_cast<long long>(s->T) * s->k > 0x7fff0000ll || static_cast<long long>(s->M_cap) > 0x7fff0000ll)
    return TEMPO_ERR_UNSUPPORTED;
  if (dispatch_smem_bytes(s->E, s->R_max, s->G_max) > 220 * 1024) return TEMPO_ERR_UNSUPPORTED;
  if (dispatch_sampled_smem_bytes(s->E, s->R_max, s->G_max) > 220 * 1024) return TEMPO_ERR_UNSUPPORTED;
  return TEMPO_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn resolve_encode_fn() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return reinterpret_cast<EncodeTiledFn>(ptr);
  return nullptr;
}

static EncodeTiledFn encode_fn() {
  // A pure host-side driver routine, looked up once; the initialisation of a function-local static
  // is thread-safe, so concurrent first calls from several threads are fine.
  static const EncodeTiledFn fn = resolve_encode_fn();
  return fn;
}

// u8 matrix [rows, cols] row-major, box = 128 columns x box_rows rows, 128-byte swizzle.
static bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols};
  const cuuint32_t box[2] = {128, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scale bytes per token of the per-token quantised activations: one per 128 columns, rounded up to 4.
static int token_sf_stride(int d) { return 4 * (((d / 128) + 3) / 4); }

static int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return n;
}

// run_mask bit 0: gate/up tiles, bit 1: down tiles.  Buffers a side does not use may be NULL.
static int launch_ffn_host(int run_mask, const tempo_shape* s, const void* a_q, const uint8_t* a_sf, const void* packed,
                           const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y,
                           uint32_t* status, void* workspace, cudaStream_t stream, int max_m = 0,
                           const int32_t* inst_count = nullptr, unsigned long long wait_ns = kDefaultWaitNs,
                           const uint8_t* x_q = nullptr, const uint8_t* x_sf = nullptr, const int32_t* row_pair = nullptr) {
  const PackLayout L = pack_layout(s->G_max, s->d, s->f);
  const uint8_t* blob = static_cast<const uint8_t*>(packed);
  const int sms = sm_count();
  if (sms <= 0) return TEMPO_ERR_CUDA;
  CUtensorMap tmA1, tmA2, tmY;
  // a side that does not run still needs a well-formed map; point it at a buffer that exists
  const bool gather = x_q != nullptr;              // gate/up rows fetched from the per-token buffers: no a_q
  if (!make_map(&tmA1, (run_mask & 1) && !gather ? a_q : h_q, s->M_cap, (run_mask & 1) && !gather ? s->d : s->f, 128))
    return TEMPO_ERR_CUDA;
  if (!make_map(&tmA2, h_q, s->M_cap, s->f, 128)) return TEMPO_ERR_CUDA;
  // Y stores: 32-row x 128-byte boxes (bf16 seen as bytes: 2d per row)
  if (!make_map(&tmY, (run_mask & 2) ? y : h_q, s->M_cap, (run_mask & 2) ? 2ull * s->d : s->f, 32)) return TEMPO_ERR_CUDA;
  FfnParams p{};
  p.side[0] = GemmSide{s->d / 128, L.J1, L.NT1, blob + L.off_w13, a_sf, blob + L.off_sf13};
  p.side[1] = GemmSide{s->f / 128, L.J2, L.NT2, blob + L.off_w2, h_sf, blob + L.off_sf2};
  p.run_mask = run_mask;
  p.G_max = s->G_max;
  p.M_cap = s->M_cap;
  p.d = s->d;
  p.f = s->f;
  p.J_h = L.J2;
  p.inst_off = inst_off;
  p.m_pad = m_pad;
  p.stride_tiles = max_m / 128;
  p.inst_count = inst_count;
  p.h_q = static_cast<uint8_t*>(h_q);
  p.h_sf = h_sf;
  p.y = static_cast<__nv_bfloat16*>(y);
  p.ready = static_cast<int32_t*>(workspace);
  p.done = p.ready ? p.ready + s->M_cap / 128 : nullptr;
  p.status = status;
  p.wait_ns = wait_ns;
  if (gather) {
    p.x_q = x_q;
    p.x_sf = x_sf;
    p.row_pair = row_pair;
    p.x_sf_stride = token_sf_stride(s->d);
    p.k = s->k;
    p.T = s->T;
    return launch_ffn_gather(tmA2, tmY, p, sms, stream) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
  }
  return launch_ffn(tmA1, tmA2, tmY, p, sms, stream) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

// ---- scratch for tempo_grouped_ffn_static ---------------------------------------------------------
// The H-ready / down-seen counters of the fused FFN kernel, two int32 per 128-row tile, for callers
// that cannot hand in a scratch buffer of their own.  Lives in every GPU that loads the library
// (128 KB) until the process ends.  The name is a host-side handle here: the device address is
// looked up once per device with cudaGetSymbolAddress and cached.
constexpr int kStaticMaxTiles = 16384;                       // M_cap <= 128 * 16384 = 2,097,152 rows
static __device__ __align__(256) int32_t g_ffn_scratch[2 * kStaticMaxTiles];
constexpr int kMaxDevices = 64;
static std::atomic<int32_t*> g_ffn_scratch_addr[kMaxDevices];   // zero-initialised; every writer stores the same value

static int32_t* static_scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int32_t* addr = g_ffn_scratch_addr[dev].load(std::memory_order_acquire);
  if (addr == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_ffn_scratch) != cudaSuccess || ptr == nullptr) return nullptr;
    addr = static_cast<int32_t*>(ptr);
    g_ffn_scratch_addr[dev].store(addr, std::memory_order_release);
  }
  return addr;
}

}  // namespace tempo

using namespace tempo;

extern "C" {

int tempo_version(void) { return 1; }

const char* tempo_status_string(int code) {
  switch (code) {
    case TEMPO_OK: return "ok";
    case TEMPO_ERR_NULL: return "a required pointer is NULL";
    case TEMPO_ERR_SHAPE: return "a size is not positive or not a multiple of 128";
    case TEMPO_ERR_UNSUPPORTED: return "a size exceeds a documented limit";
    case TEMPO_ERR_CUDA: return "a CUDA call failed";
    default: return "unknown code";
  }
}

int tempo_m_cap_bound(const tempo_shape* s, int32_t* m_cap) {
  if (s == nullptr || m_cap == nullptr) return TEMPO_ERR_NULL;
  if (s->T <= 0 || s->k <= 0 || s->G_max <= 0) return TEMPO_ERR_SHAPE;
  const long long v = ((static_cast<long long>(s->T) * s->k + 127) / 128) * 128 + 128ll * s->G_max;
  if (v > 0x7fff0000ll) return TEMPO_ERR_UNSUPPORTED;
  *m_cap = static_cast<int32_t>(v);
  return TEMPO_OK;
}

int tempo_sf_bytes(int32_t rows, int32_t cols, size_t* bytes) {
  if (bytes == nullptr) return TEMPO_ERR_NULL;
  if (rows <= 0 || cols <= 0 || rows % 128 || cols % 128) return TEMPO_ERR_SHAPE;
  *bytes = static_cast<size_t>(rows / 128) * (((cols / 128) + 3) / 4) * 512;
  return TEMPO_OK;
}

int tempo_workspace_bytes(const tempo_shape* s, size_t* bytes) {
  if (bytes == nullptr) return TEMPO_ERR_NULL;
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  *bytes = ffn_workspace_bytes(s->M_cap);
  return TEMPO_OK;
}

int tempo_packed_weight_bytes(const tempo_shape* s, size_t* bytes) {
  if (bytes == nullptr) return TEMPO_ERR_NULL;
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  *bytes = pack_layout(s->G_max, s->d, s->f).total;
  return TEMPO_OK;
}

int tempo_pack_weights(const tempo_shape* s, const void* w13_q, const float* w13_s, const void* w2_q,
                       const float* w2_s, void* packed, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!w13_q || !w13_s || !w2_q || !w2_s || !packed || !status) return TEMPO_ERR_NULL;
  return launch_pack(s->G_max, s->d, s->f, static_cast<const uint8_t*>(w13_q), w13_s,
                     static_cast<const uint8_t*>(w2_q), w2_s, static_cast<uint8_t*>(packed), status,
                     static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_count_dispatch(const tempo_shape* s, const int32_t* topk_ids, const int32_t* n_valid,
                         const int32_t* replica_map, const int32_t* quota, uint32_t* cum_counts,
                         int32_t* counts, int32_t* inst_count, int32_t* inst_off, int32_t* pair_row,
                         int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!topk_ids || !replica_map || !quota || !counts || !inst_count || !inst_off || !pair_row || !row_pair ||
      !tile_inst || !m_pad || !status)
    return TEMPO_ERR_NULL;
  DispatchParams p{s->T, s->k, s->E, s->G_max, s->R_max, s->M_cap, topk_ids, n_valid, replica_map, quota,
                   cum_counts, counts, inst_count, inst_off, pair_row, row_pair, tile_inst, m_pad, status};
  return launch_count_dispatch(p, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_count_dispatch_sampled(const tempo_shape* s, const int32_t* topk_ids, const int32_t* n_valid,
                                 const int32_t* replica_map, const float* table, uint64_t seed, uint32_t layer,
                                 uint32_t* cum_counts, int32_t* counts, int32_t* inst_count, int32_t* inst_off,
                                 int32_t* pair_row, int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad,
                                 uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!topk_ids || !replica_map || !table || !counts || !inst_count || !inst_off || !pair_row || !row_pair ||
      !tile_inst || !m_pad || !status)
    return TEMPO_ERR_NULL;
  SampledParams p{s->T, s->k, s->E, s->G_max, s->R_max, s->M_cap, topk_ids, n_valid, replica_map, table,
                  static_cast<unsigned long long>(seed), layer, cum_counts, counts, inst_count, inst_off, pair_row,
                  row_pair, tile_inst, m_pad, status};
  return launch_count_dispatch_sampled(p, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_permute_pad(const tempo_shape* s, const void* x_bf16, const int32_t* row_pair, const int32_t* pair_row,
                      const int32_t* m_pad, void* a_q, uint8_t* a_sf, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!x_bf16 || !row_pair || !m_pad || !a_q || !a_sf || !status) return TEMPO_ERR_NULL;
  PermuteParams p{s->k, s->d, s->M_cap, static_cast<const __nv_bfloat16*>(x_bf16), row_pair, s->T, pair_row, nullptr, m_pad,
                  static_cast<uint8_t*>(a_q), a_sf};
  return launch_permute_pad(p, sm_count(), static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_ffn_gate_up(const tempo_shape* s, const void* a_q, const uint8_t* a_sf, const void* packed,
                      const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, uint32_t* status,
                      void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!a_q || !a_sf || !packed || !inst_off || !m_pad || !h_q || !h_sf || !status) return TEMPO_ERR_NULL;
  return launch_ffn_host(1, s, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, nullptr, status, nullptr,
                         static_cast<cudaStream_t>(stream));
}

int tempo_ffn_down(const tempo_shape* s, const void* h_q, const uint8_t* h_sf, const void* packed,
                   const int32_t* inst_off, const int32_t* m_pad, void* y_bf16, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!h_q || !h_sf || !packed || !inst_off || !m_pad || !y_bf16 || !status) return TEMPO_ERR_NULL;
  return launch_ffn_host(2, s, nullptr, nullptr, packed, inst_off, m_pad, const_cast<void*>(h_q),
                         const_cast<uint8_t*>(h_sf), y_bf16, status, nullptr, static_cast<cudaStream_t>(stream));
}

int tempo_grouped_ffn(const tempo_shape* s, const void* a_q, const uint8_t* a_sf, const void* packed,
                      const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                      uint32_t* status, void* workspace, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!a_q || !a_sf || !packed || !inst_off || !m_pad || !h_q || !h_sf || !y_bf16 || !status || !workspace)
    return TEMPO_ERR_NULL;
  return launch_ffn_host(3, s, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace,
                         static_cast<cudaStream_t>(stream));
}

int tempo_token_sf_bytes(const tempo_shape* s, size_t* bytes) {
  if (bytes == nullptr) return TEMPO_ERR_NULL;
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  *bytes = static_cast<size_t>(s->T) * token_sf_stride(s->d);
  return TEMPO_OK;
}

int tempo_quantize_tokens(const tempo_shape* s, const void* x_bf16, const int32_t* n_valid, void* x_q, uint8_t* x_sf,
                          uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!x_bf16 || !x_q || !x_sf || !status) return TEMPO_ERR_NULL;
  QuantizeParams p{s->T, s->d, token_sf_stride(s->d), static_cast<const __nv_bfloat16*>(x_bf16), n_valid,
                   static_cast<uint8_t*>(x_q), x_sf};
  return launch_quantize_tokens(p, sm_count(), static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_grouped_ffn_gather(const tempo_shape* s, const void* x_q, const uint8_t* x_sf, const int32_t* row_pair,
                             const void* packed, const int32_t* inst_off, const int32_t* m_pad, void* h_q,
                             uint8_t* h_sf, void* y_bf16, uint32_t* status, void* workspace, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!x_q || !x_sf || !row_pair || !packed || !inst_off || !m_pad || !h_q || !h_sf || !y_bf16 || !status || !workspace)
    return TEMPO_ERR_NULL;
  return launch_ffn_host(3, s, nullptr, nullptr, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace,
                         static_cast<cudaStream_t>(stream), 0, nullptr, kDefaultWaitNs, static_cast<const uint8_t*>(x_q),
                         x_sf, row_pair);
}

int tempo_grouped_ffn_bounded(const tempo_shape* s, const void* a_q, const uint8_t* a_sf, const void* packed,
                              const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                              uint32_t* status, void* workspace, uint64_t wait_limit_ns, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!a_q || !a_sf || !packed || !inst_off || !m_pad || !h_q || !h_sf || !y_bf16 || !status || !workspace)
    return TEMPO_ERR_NULL;
  if (wait_limit_ns == 0) return TEMPO_ERR_SHAPE;
  return launch_ffn_host(3, s, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, workspace,
                         static_cast<cudaStream_t>(stream), 0, nullptr, wait_limit_ns);
}

int tempo_grouped_ffn_static(const tempo_shape* s, const void* a_q, const uint8_t* a_sf, const void* packed,
                             const int32_t* inst_off, const int32_t* m_pad, void* h_q, uint8_t* h_sf, void* y_bf16,
                             uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!a_q || !a_sf || !packed || !inst_off || !m_pad || !h_q || !h_sf || !y_bf16 || !status) return TEMPO_ERR_NULL;
  if (s->M_cap / 128 > kStaticMaxTiles) return TEMPO_ERR_UNSUPPORTED;      // beyond the built-in scratch
  int32_t* scratch = static_scratch_for_current_device();
  if (scratch == nullptr) return TEMPO_ERR_CUDA;
  // the array keeps whatever the last call left (normally zeros; not after a timed-out call): start clean
  if (cudaMemsetAsync(scratch, 0, 2 * sizeof(int32_t) * static_cast<size_t>(s->M_cap / 128),
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return TEMPO_ERR_CUDA;
  return launch_ffn_host(3, s, a_q, a_sf, packed, inst_off, m_pad, h_q, h_sf, y_bf16, status, scratch,
                         static_cast<cudaStream_t>(stream));
}

// ---- masked layout ------------------------------------------------------------------------------------
static int check_masked(const tempo_shape* s, int32_t max_m) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (max_m <= 0 || max_m % 128 != 0) return TEMPO_ERR_SHAPE;
  if (static_cast<long long>(s->G_max) * max_m > s->M_cap) return TEMPO_ERR_SHAPE;
  return TEMPO_OK;
}

int tempo_count_dispatch_masked(const tempo_shape* s, int32_t max_m, const int32_t* topk_ids, const int32_t* n_valid,
                                const int32_t* replica_map, const int32_t* quota, uint32_t* cum_counts,
                                int32_t* counts, int32_t* inst_count, int32_t* inst_off, int32_t* pair_row,
                                int32_t* row_pair, int32_t* tile_inst, int32_t* m_pad, uint32_t* status, void* stream) {
  const int rc = check_masked(s, max_m);
  if (rc != TEMPO_OK) return rc;
  if (!topk_ids || !replica_map || !quota || !counts || !inst_count || !inst_off || !pair_row || !row_pair ||
      !tile_inst || !m_pad || !status)
    return TEMPO_ERR_NULL;
  DispatchParams p{s->T, s->k, s->E, s->G_max, s->R_max, s->M_cap, topk_ids, n_valid, replica_map, quota,
                   cum_counts, counts, inst_count, inst_off, pair_row, row_pair, tile_inst, m_pad, status, max_m};
  return launch_count_dispatch(p, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_permute_pad_masked(const tempo_shape* s, const void* x_bf16, const int32_t* row_pair, const int32_t* pair_row,
                             const int32_t* tile_inst, const int32_t* m_pad, void* a_q, uint8_t* a_sf,
                             uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!x_bf16 || !row_pair || !pair_row || !tile_inst || !m_pad || !a_q || !a_sf || !status) return TEMPO_ERR_NULL;
  PermuteParams p{s->k, s->d, s->M_cap, static_cast<const __nv_bfloat16*>(x_bf16), row_pair, s->T, pair_row, tile_inst,
                  m_pad, static_cast<uint8_t*>(a_q), a_sf};
  return launch_permute_pad(p, sm_count(), static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_grouped_ffn_masked(const tempo_shape* s, int32_t max_m, const void* a_q, const uint8_t* a_sf,
                             const void* packed, const int32_t* inst_count, void* h_q, uint8_t* h_sf, void* y_bf16,
                             uint32_t* status, void* workspace, void* stream) {
  const int rc = check_masked(s, max_m);
  if (rc != TEMPO_OK) return rc;
  if (!a_q || !a_sf || !packed || !inst_count || !h_q || !h_sf || !y_bf16 || !status || !workspace) return TEMPO_ERR_NULL;
  return launch_ffn_host(3, s, a_q, a_sf, packed, nullptr, nullptr, h_q, h_sf, y_bf16, status, workspace,
                         static_cast<cudaStream_t>(stream), max_m, inst_count);
}

// ---- bf16 variant of steps 2 and 3 -------------------------------------------------------------------
int tempo_packed_weight_bytes_bf16(const tempo_shape* s, size_t* bytes) {
  if (bytes == nullptr) return TEMPO_ERR_NULL;
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  *bytes = pack_layout_bf16(s->G_max, s->d, s->f).total;
  return TEMPO_OK;
}

int tempo_pack_weights_bf16(const tempo_shape* s, const void* w13_bf16, const void* w2_bf16, void* packed, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!w13_bf16 || !w2_bf16 || !packed) return TEMPO_ERR_NULL;
  return launch_pack_bf16(s->G_max, s->d, s->f, static_cast<const __nv_bfloat16*>(w13_bf16),
                          static_cast<const __nv_bfloat16*>(w2_bf16), static_cast<uint8_t*>(packed),
                          static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_permute_pad_bf16(const tempo_shape* s, const void* x_bf16, const int32_t* row_pair, const int32_t* m_pad,
                           void* a_bf16, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!x_bf16 || !row_pair || !m_pad || !a_bf16 || !status) return TEMPO_ERR_NULL;
  PermuteParams p{s->k, s->d, s->M_cap, static_cast<const __nv_bfloat16*>(x_bf16), row_pair, s->T, nullptr, nullptr, m_pad, nullptr, nullptr};
  return launch_permute_pad_bf16(p, static_cast<__nv_bfloat16*>(a_bf16), sm_count(), static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

int tempo_grouped_ffn_bf16(const tempo_shape* s, const void* a_bf16, const void* packed, const int32_t* inst_off,
                           const int32_t* m_pad, void* h_bf16, void* y_bf16, uint32_t* status, void* workspace,
                           void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!a_bf16 || !packed || !inst_off || !m_pad || !h_bf16 || !y_bf16 || !status || !workspace) return TEMPO_ERR_NULL;
  const PackLayout L = pack_layout_bf16(s->G_max, s->d, s->f);
  const uint8_t* blob = static_cast<const uint8_t*>(packed);
  const int sms = sm_count();
  if (sms <= 0) return TEMPO_ERR_CUDA;
  CUtensorMap tmA1, tmA2, tmY;    // bf16 matrices seen as bytes: 2d / 2f per row
  if (!make_map(&tmA1, a_bf16, s->M_cap, 2ull * s->d, 128)) return TEMPO_ERR_CUDA;
  if (!make_map(&tmA2, h_bf16, s->M_cap, 2ull * s->f, 128)) return TEMPO_ERR_CUDA;
  if (!make_map(&tmY, y_bf16, s->M_cap, 2ull * s->d, 32)) return TEMPO_ERR_CUDA;
  FfnParams p{};
  p.side[0] = GemmSide{s->d / 64, 0, L.NT1, blob + L.off_w13, nullptr, nullptr};
  p.side[1] = GemmSide{s->f / 64, 0, L.NT2, blob + L.off_w2, nullptr, nullptr};
  p.run_mask = 3;
  p.G_max = s->G_max;
  p.M_cap = s->M_cap;
  p.d = s->d;
  p.f = s->f;
  p.inst_off = inst_off;
  p.m_pad = m_pad;
  p.h_q = static_cast<uint8_t*>(h_bf16);
  p.y = static_cast<__nv_bfloat16*>(y_bf16);
  p.ready = static_cast<int32_t*>(workspace);
  p.done = p.ready + s->M_cap / 128;
  p.status = status;
  p.wait_ns = kDefaultWaitNs;
  return launch_ffn_bf16(tmA1, tmA2, tmY, p, sms, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK
                                                                                                         : TEMPO_ERR_CUDA;
}

int tempo_unpermute_combine(const tempo_shape* s, const void* y_bf16, const int32_t* pair_row, const float* topk_w,
                            const int32_t* n_valid, void* out_bf16, uint32_t* status, void* stream) {
  const int rc = check_shape(s);
  if (rc != TEMPO_OK) return rc;
  if (!y_bf16 || !pair_row || !topk_w || !out_bf16 || !status) return TEMPO_ERR_NULL;
  CombineParams p{s->T, s->k, s->d, static_cast<const __nv_bfloat16*>(y_bf16), pair_row, topk_w, n_valid,
                  static_cast<__nv_bfloat16*>(out_bf16)};
  return launch_combine(p, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TEMPO_OK : TEMPO_ERR_CUDA;
}

}  // extern "C"
