// C ABI of the SparseD attention library: argument validation, tensor-map construction,
// workspace layout and kernel dispatch. Declarations and contracts are in sparsed.h.
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/sparsed.h"
#include "internal.h"

namespace {

using namespace sparsed;

thread_local int32_t g_last_cuda_error = 0;

sparsed_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int32_t>(e);
  return SPARSED_ERR_CUDA;
}

// ---- driver entry point for tensor-map encoding (no link-time dependency on libcuda) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(p);
    }
  });
  return fn;
}

// Host-side cache of encoded tensor maps. A map depends only on (base pointer, extents, strides,
// box), not on the tensor's contents, so a denoising loop that calls with the same buffers every
// step encodes each map once. Per thread (no locking), direct-mapped, 32 entries.
struct TensorMapKey {
  const void* base;
  int64_t strides[3];
  int32_t batch, heads, seq_len, box_rows;
  bool operator==(const TensorMapKey& o) const {
    return base == o.base && strides[0] == o.strides[0] && strides[1] == o.strides[1] && strides[2] == o.strides[2] &&
           batch == o.batch && heads == o.heads && seq_len == o.seq_len && box_rows == o.box_rows;
  }
};
struct TensorMapSlot {
  TensorMapKey key;
  CUtensorMap map;
  bool valid;
};
constexpr int kTensorMapSlots = 32;
thread_local TensorMapSlot g_tensor_maps[kTensorMapSlots] = {};

uint32_t tensor_map_slot(const TensorMapKey& k) {
  uint64_t h = reinterpret_cast<uintptr_t>(k.base) >> 4;
  h = h * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(k.strides[1]);
  h = h * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(k.strides[2]);
  h = h * 0x9E3779B97F4A7C15ull + (static_cast<uint64_t>(k.seq_len) << 8 | static_cast<uint64_t>(k.box_rows));
  h = h * 0x9E3779B97F4A7C15ull + (static_cast<uint64_t>(k.heads) << 16 | static_cast<uint64_t>(k.batch));
  return static_cast<uint32_t>(h >> 40) % kTensorMapSlots;
}

// bf16 [B,H,L,128] tensor with element strides (batch, head, token); box = 64 x rows, 128B swizzle.
sparsed_status make_tensor_map(CUtensorMap* out, const void* base, int batch, int heads, int seq_len,
                               const int64_t strides[3], int box_rows) {
  TensorMapKey key{base, {strides[0], strides[1], strides[2]}, batch, heads, seq_len, box_rows};
  TensorMapSlot& slot = g_tensor_maps[tensor_map_slot(key)];
  if (slot.valid && slot.key == key) {
    *out = slot.map;
    return SPARSED_OK;
  }
  EncodeTiledFn enc = encode_tiled_fn();
  if (enc == nullptr) return cuda_fail(cudaErrorNotSupported);
  cuuint64_t dims[4] = {128, static_cast<cuuint64_t>(seq_len), static_cast<cuuint64_t>(heads),
                        static_cast<cuuint64_t>(batch)};
  cuuint64_t gstrides[3] = {static_cast<cuuint64_t>(strides[2]) * 2, static_cast<cuuint64_t>(strides[1]) * 2,
                            static_cast<cuuint64_t>(strides[0]) * 2};
  cuuint32_t box[4] = {64, static_cast<cuuint32_t>(box_rows), 1, 1};
  cuuint32_t elem[4] = {1, 1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, gstrides, box, elem,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = static_cast<int32_t>(r);
    return SPARSED_ERR_CUDA;
  }
  slot.key = key;
  slot.map = *out;
  slot.valid = true;
  return SPARSED_OK;
}

struct Resolved {
  int64_t q[3], k[3], v[3], o[3];
  float scale_log2;
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

// The workspace holds the status word (atomics) and fp32 arrays the kernels read with 16-byte loads.
sparsed_status check_ws(const void* ws, size_t ws_bytes, size_t need) {
  if (ws == nullptr || ws_bytes < need) return SPARSED_ERR_WORKSPACE;
  return aligned16(ws) ? SPARSED_OK : SPARSED_ERR_ALIGNMENT;
}

void default_strides(const int64_t in[3], int heads, int seq_len, int64_t out[3]) {
  if (in[0] == 0 && in[1] == 0 && in[2] == 0) {
    out[2] = 128;
    out[1] = static_cast<int64_t>(seq_len) * 128;
    out[0] = out[1] * heads;
  } else {
    out[0] = in[0];
    out[1] = in[1];
    out[2] = in[2];
  }
}

sparsed_status check_arch() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  static std::atomic<int> cached_major[64];  // 0 = not looked up yet
  int major = (dev >= 0 && dev < 64) ? cached_major[dev].load(std::memory_order_relaxed) : 0;
  if (major == 0) {
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev >= 0 && dev < 64) cached_major[dev].store(major, std::memory_order_relaxed);
  }
  return major == 10 ? SPARSED_OK : SPARSED_ERR_ARCH;
}

// CTAs of the attention kernel that are resident on the current device at once (two per SM), cached per
// device; 0 if the SM count cannot be read (the kernel then gets one CTA per query tile).
int attn_max_ctas() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  static std::atomic<int> cached[64];
  int n = (dev >= 0 && dev < 64) ? cached[dev].load(std::memory_order_relaxed) : 0;
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64) cached[dev].store(n, std::memory_order_relaxed);
  }
  return 2 * n;
}

sparsed_status check_shape(const sparsed_shape* s, bool need_v_o, Resolved* r) {
  if (s == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (s->batch < 1 || s->heads_q < 1 || s->heads_kv < 1 || s->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
  if (s->heads_q % s->heads_kv != 0) return SPARSED_ERR_INVALID_ARG;
  if (s->head_dim != 128) return SPARSED_ERR_UNSUPPORTED;
  if (!(s->softmax_scale >= 0.f) || !std::isfinite(s->softmax_scale)) return SPARSED_ERR_INVALID_ARG;
  default_strides(s->q_strides, s->heads_q, s->seq_len, r->q);
  default_strides(s->k_strides, s->heads_kv, s->seq_len, r->k);
  default_strides(s->v_strides, s->heads_kv, s->seq_len, r->v);
  default_strides(s->o_strides, s->heads_q, s->seq_len, r->o);
  const int64_t* sets[4] = {r->q, r->k, r->v, r->o};
  for (int t = 0; t < (need_v_o ? 4 : 2); ++t) {
    for (int i = 0; i < 3; ++i) {
      if (sets[t][i] <= 0) return SPARSED_ERR_INVALID_ARG;
      if (sets[t][i] % 8 != 0) return SPARSED_ERR_ALIGNMENT;
    }
    if (sets[t][2] < 128) return SPARSED_ERR_INVALID_ARG;
  }
  const float scale = s->softmax_scale == 0.f ? 1.0f / std::sqrt(static_cast<float>(s->head_dim)) : s->softmax_scale;
  r->scale_log2 = scale * 1.44269504088896341f;
  return SPARSED_OK;
}

sparsed_status kept_counts(const sparsed_select_params* sp, int nb, int* pb, int* k_pre, int* k_gen) {
  if (sp == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (sp->block_size != 32 && sp->block_size != 64 && sp->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (!(sp->keep_ratio > 0.0) || !(sp->keep_ratio <= 1.0)) return SPARSED_ERR_INVALID_ARG;
  if (sp->rounding != 0 && sp->rounding != 1) return SPARSED_ERR_INVALID_ARG;
  if (sp->prefill_len < 0) return SPARSED_ERR_INVALID_ARG;
  if (sp->prefill_len % sp->block_size != 0) return SPARSED_ERR_ALIGNMENT;
  const int p_blocks = sp->prefill_len / sp->block_size;
  if (p_blocks > nb) return SPARSED_ERR_INVALID_ARG;
  auto kept = [&](int n) -> int {
    if (n <= 0) return 0;
    const double x = sp->keep_ratio * n;
    long long kk = sp->rounding == 0 ? static_cast<long long>(std::ceil(x - 1e-6))
                                     : static_cast<long long>(std::floor(x + 1e-6));
    if (kk < 1) kk = 1;
    if (kk > n) kk = n;
    return static_cast<int>(kk);
  };
  *pb = p_blocks;
  *k_pre = kept(p_blocks);
  *k_gen = kept(nb - p_blocks);
  return SPARSED_OK;
}

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Whether the switch step can select from the row statistics of its own full-attention pass.
bool step_uses_stats(const sparsed_shape* shape, const sparsed_select_params* params) {
  return shape->seq_len / params->block_size <= pool_select_max_blocks();
}

// Checks the caller's pattern buffers against the number of rows and kept blocks per row and
// fills in the host-side fields of `out`.
sparsed_status prepare_pattern(sparsed_pattern* out, int batch, int heads_q, int nb, int block_size, int k_total) {
  if (out == nullptr || out->row_ptr == nullptr || out->col_idx == nullptr) return SPARSED_ERR_PATTERN;
  if (!aligned4(out->row_ptr) || !aligned4(out->col_idx)) return SPARSED_ERR_ALIGNMENT;
  if (nb > 16384) return SPARSED_ERR_UNSUPPORTED;
  const int64_t rows = static_cast<int64_t>(batch) * heads_q * nb;
  const int64_t nnz = rows * k_total;
  if (rows >= INT32_MAX || nnz >= INT32_MAX) return SPARSED_ERR_UNSUPPORTED;
  if (out->col_capacity < nnz) return SPARSED_ERR_PATTERN;
  out->nnz = nnz;
  out->block_size = block_size;
  out->num_blocks = nb;
  out->batch = batch;
  out->heads_q = heads_q;
  return SPARSED_OK;
}

sparsed_status run_topk(const float* scores, int batch, int heads_q, int nb, int block_size, int pb, int k_pre,
                        int k_gen, sparsed_pattern* out, cudaStream_t stream) {
  sparsed_status st = prepare_pattern(out, batch, heads_q, nb, block_size, k_pre + k_gen);
  if (st != SPARSED_OK) return st;
  TopkParams tp;
  tp.scores = scores;
  tp.row_ptr = out->row_ptr;
  tp.col_idx = out->col_idx;
  tp.rows = batch * heads_q * nb;
  tp.nb = nb;
  tp.pb = pb;
  tp.k_pre = k_pre;
  tp.k_gen = k_gen;
  cudaError_t e = launch_topk_csr(tp, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return SPARSED_OK;
}

}  // namespace

extern "C" {

const char* sparsed_status_string(sparsed_status status) {
  switch (status) {
    case SPARSED_OK: return "ok";
    case SPARSED_ERR_INVALID_ARG: return "invalid argument";
    case SPARSED_ERR_UNSUPPORTED: return "unsupported configuration";
    case SPARSED_ERR_ALIGNMENT: return "alignment or divisibility requirement not met";
    case SPARSED_ERR_WORKSPACE: return "workspace missing or too small";
    case SPARSED_ERR_PATTERN: return "pattern invalid or too small";
    case SPARSED_ERR_ARCH: return "device is not compute capability 10.x";
    case SPARSED_ERR_CUDA: return "CUDA error";
    case SPARSED_ERR_DEVICE_TIMEOUT: return "device-side wait ran out";
  }
  return "unknown status";
}

int32_t sparsed_last_cuda_error(void) { return g_last_cuda_error; }

int32_t sparsed_switch_step(int32_t total_steps, double skip) {
  if (total_steps < 1 || !(skip >= 0.0) || !(skip <= 1.0)) return -1;
  long long s = static_cast<long long>(std::floor(static_cast<double>(total_steps) * skip + 1e-9));
  if (s < 1) s = 1;
  if (s > total_steps) s = total_steps;
  return static_cast<int32_t>(s);
}

int32_t sparsed_schedule_mode(int32_t step_1based, int32_t total_steps, double skip) {
  const int32_t s = sparsed_switch_step(total_steps, skip);
  if (s < 0 || step_1based < 1 || step_1based > total_steps) return -1;
  if (step_1based < s) return SPARSED_MODE_FULL;
  if (step_1based == s) return SPARSED_MODE_FULL_AND_SELECT;
  return SPARSED_MODE_SPARSE;
}

sparsed_status sparsed_kept_per_row(const sparsed_select_params* params, int32_t seq_len, int32_t* k_pre,
                                    int32_t* k_gen) {
  if (params == nullptr || k_pre == nullptr || k_gen == nullptr || seq_len < 1) return SPARSED_ERR_INVALID_ARG;
  if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
  int pb = 0, a = 0, b = 0;
  sparsed_status st = kept_counts(params, seq_len / params->block_size, &pb, &a, &b);
  if (st != SPARSED_OK) return st;
  *k_pre = a;
  *k_gen = b;
  return SPARSED_OK;
}

sparsed_status sparsed_workspace_bytes(int32_t op, const sparsed_shape* shape, const sparsed_select_params* params,
                                       size_t* out_bytes) {
  if (out_bytes == nullptr) return SPARSED_ERR_INVALID_ARG;
  switch (op) {
    case SPARSED_OP_ATTN_FULL:
    case SPARSED_OP_ATTN_SPARSE:
    case SPARSED_OP_SELECT_FROM_SCORES:
    case SPARSED_OP_PATTERN_VALIDATE:
      *out_bytes = SPARSED_STATUS_BYTES;
      return SPARSED_OK;
    case SPARSED_OP_SELECT_PATTERN: {
      if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
      if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
      if (shape->batch < 1 || shape->heads_q < 1 || shape->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
      if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
      const size_t nb = static_cast<size_t>(shape->seq_len / params->block_size);
      const size_t bh = static_cast<size_t>(shape->batch) * shape->heads_q;
      *out_bytes = SPARSED_STATUS_BYTES + round_up(bh * nb * nb * 4, 256) +
                   round_up(bh * static_cast<size_t>(shape->seq_len) * 4, 256);
      return SPARSED_OK;
    }
    case SPARSED_OP_SELECT_POOLED_QK: {
      if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
      if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
      if (shape->batch < 1 || shape->heads_q < 1 || shape->heads_kv < 1 || shape->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
      if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
      *out_bytes = SPARSED_STATUS_BYTES +
                   pooled_qk_means_bytes(shape->batch, shape->heads_q, shape->heads_kv, shape->seq_len / params->block_size);
      return SPARSED_OK;
    }
    case SPARSED_OP_ATTENTION_STEP: {
      if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
      if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
      if (shape->batch < 1 || shape->heads_q < 1 || shape->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
      if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
      const size_t nb = static_cast<size_t>(shape->seq_len / params->block_size);
      const size_t bh = static_cast<size_t>(shape->batch) * shape->heads_q;
      const size_t lse_bytes = round_up(bh * static_cast<size_t>(shape->seq_len) * 4, 256);
      if (step_uses_stats(shape, params)) {
        size_t stats = 0;
        sparsed_status st = sparsed_tile_stats_bytes(shape, params->block_size, &stats);
        if (st != SPARSED_OK) return st;
        *out_bytes = SPARSED_STATUS_BYTES + lse_bytes + stats;
      } else {
        *out_bytes = SPARSED_STATUS_BYTES + round_up(bh * nb * nb * 4, 256) + lse_bytes;
      }
      return SPARSED_OK;
    }
    default:
      return SPARSED_ERR_INVALID_ARG;
  }
}

sparsed_status sparsed_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream) {
  sparsed_status st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES);
  if (st != SPARSED_OK) return st;
  cudaError_t e = cudaMemsetAsync(ws, 0, SPARSED_STATUS_BYTES, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

// Which dense kernel runs. The pass that also records row statistics has one kernel, whose MMAs span CTA
// pairs (attention_dense_pair.cu). The plain pass runs it from 16k tokens on (measured 3-4 % faster there) and
// the single-CTA kernel (attention.cu) below that, where a cluster's short life makes the pair kernel no
// faster under sustained load and slower per launch. The environment variable SPARSED_DENSE_KERNEL (read once)
// sends every plain pass to one of them, `pair` or `single`, for A/B measurements and tests.
static bool dense_pair_kernel(bool with_stats, int seq_len) {
  static const int forced = [] {
    const char* v = std::getenv("SPARSED_DENSE_KERNEL");
    if (v != nullptr && std::strcmp(v, "pair") == 0) return 1;
    if (v != nullptr && std::strcmp(v, "single") == 0) return 0;
    return -1;
  }();
  if (with_stats) return true;
  return forced >= 0 ? forced == 1 : seq_len >= 16384;
}

static sparsed_status attn_full_impl(const sparsed_shape* shape, const void* q, const void* k, const void* v, void* o,
                                     float* lse_or_null, float* tile_lse_or_null, int stat_keys, void* ws,
                                     size_t ws_bytes, void* cuda_stream) {
  Resolved rs;
  sparsed_status st = check_shape(shape, true, &rs);
  if (st != SPARSED_OK) return st;
  if (q == nullptr || k == nullptr || v == nullptr || o == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return SPARSED_ERR_ALIGNMENT;
  if (!aligned16(lse_or_null) || !aligned16(tile_lse_or_null)) return SPARSED_ERR_ALIGNMENT;
  if ((st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES)) != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  const bool pair = dense_pair_kernel(tile_lse_or_null != nullptr, shape->seq_len);
  CUtensorMap tq, tk, tv, to;
  if ((st = make_tensor_map(&tq, q, shape->batch, shape->heads_q, shape->seq_len, rs.q, 128)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&to, o, shape->batch, shape->heads_q, shape->seq_len, rs.o, 128)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&tk, k, shape->batch, shape->heads_kv, shape->seq_len, rs.k, pair ? 32 : 64)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&tv, v, shape->batch, shape->heads_kv, shape->seq_len, rs.v, 64)) != SPARSED_OK) return st;
  AttnParams p;
  p.o = o;
  p.o_stride_b = rs.o[0];
  p.o_stride_h = rs.o[1];
  p.o_stride_t = rs.o[2];
  p.lse = lse_or_null;
  p.tile_lse = tile_lse_or_null;
  p.stat_keys = stat_keys;
  p.slow_path_events = reinterpret_cast<unsigned long long*>(static_cast<uint8_t*>(ws) + 32);
  p.seq_len = shape->seq_len;
  p.heads_q = shape->heads_q;
  p.group = shape->heads_q / shape->heads_kv;
  p.num_q_tiles = (shape->seq_len + 127) / 128;
  p.num_blocks = 0;
  p.num_items = shape->batch * shape->heads_q * p.num_q_tiles;
  p.max_ctas = 0;   // dense: one CTA per query tile (running on into further tiles measured 1-2 % slower here)
  p.scale_log2 = rs.scale_log2;
  p.row_ptr = nullptr;
  p.col_idx = nullptr;
  p.col_capacity = 0;
  p.status = static_cast<DeviceStatus*>(ws);
  cudaError_t e = pair ? launch_attn_dense_pair(tq, tk, tv, to, p, static_cast<cudaStream_t>(cuda_stream))
                      : launch_attn_dense(tq, tk, tv, to, p, shape->batch, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

sparsed_status sparsed_attn_full(const sparsed_shape* shape, const void* q, const void* k, const void* v, void* o,
                                 float* lse_or_null, void* ws, size_t ws_bytes, void* cuda_stream) {
  return attn_full_impl(shape, q, k, v, o, lse_or_null, nullptr, 64, ws, ws_bytes, cuda_stream);
}

sparsed_status sparsed_tile_stats_bytes(const sparsed_shape* shape, int32_t block_size, size_t* out_bytes) {
  if (shape == nullptr || out_bytes == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (shape->batch < 1 || shape->heads_q < 1 || shape->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
  if (block_size != 32 && block_size != 64 && block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (shape->seq_len % block_size != 0) return SPARSED_ERR_ALIGNMENT;
  const size_t groups = static_cast<size_t>(shape->seq_len / block_size);
  const size_t q_tiles = (static_cast<size_t>(shape->seq_len) + 127) / 128;
  *out_bytes = static_cast<size_t>(shape->batch) * shape->heads_q * q_tiles * groups * 128 * 4;
  return SPARSED_OK;
}

sparsed_status sparsed_attn_full_stats(const sparsed_shape* shape, int32_t block_size, const void* q, const void* k,
                                       const void* v, void* o, float* lse, float* tile_stats, void* ws,
                                       size_t ws_bytes, void* cuda_stream) {
  if (shape == nullptr || lse == nullptr || tile_stats == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (block_size != 32 && block_size != 64 && block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (shape->seq_len >= 1 && shape->seq_len % block_size != 0) return SPARSED_ERR_ALIGNMENT;
  return attn_full_impl(shape, q, k, v, o, lse, tile_stats, block_size, ws, ws_bytes, cuda_stream);
}

sparsed_status sparsed_select_from_stats(const sparsed_shape* shape, const sparsed_select_params* params,
                                         const float* lse, const float* tile_stats, sparsed_pattern* out,
                                         float* scores_out_or_null, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (shape->batch < 1 || shape->heads_q < 1 || shape->seq_len < 1) return SPARSED_ERR_INVALID_ARG;
  if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
  const int nb = shape->seq_len / params->block_size;
  int pb = 0, k_pre = 0, k_gen = 0;
  sparsed_status st = kept_counts(params, nb, &pb, &k_pre, &k_gen);
  if (st != SPARSED_OK) return st;
  if (lse == nullptr || tile_stats == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(lse) || !aligned16(tile_stats) || !aligned16(scores_out_or_null)) return SPARSED_ERR_ALIGNMENT;
  if (nb > pool_select_max_blocks()) return SPARSED_ERR_UNSUPPORTED;
  if ((st = prepare_pattern(out, shape->batch, shape->heads_q, nb, params->block_size, k_pre + k_gen)) != SPARSED_OK)
    return st;
  if ((st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES)) != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  PoolParams pp;
  pp.tile_lse = tile_stats;
  pp.lse = lse;
  pp.scores = scores_out_or_null;
  pp.row_ptr = out->row_ptr;
  pp.col_idx = out->col_idx;
  pp.seq_len = shape->seq_len;
  pp.block_size = params->block_size;
  pp.pb = pb;
  pp.k_pre = k_pre;
  pp.k_gen = k_gen;
  pp.bh = shape->batch * shape->heads_q;
  cudaError_t e = launch_pool_select(pp, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

sparsed_status sparsed_select_pattern_pooled_qk(const sparsed_shape* shape, const sparsed_select_params* params,
                                                const void* q, const void* k, sparsed_pattern* out,
                                                float* scores_out_or_null, void* ws, size_t ws_bytes,
                                                void* cuda_stream) {
  Resolved rs;
  sparsed_status st = check_shape(shape, false, &rs);
  if (st != SPARSED_OK) return st;
  if (params == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (q == nullptr || k == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(scores_out_or_null)) return SPARSED_ERR_ALIGNMENT;
  if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
  const int nb = shape->seq_len / params->block_size;
  int pb = 0, k_pre = 0, k_gen = 0;
  if ((st = kept_counts(params, nb, &pb, &k_pre, &k_gen)) != SPARSED_OK) return st;
  if (nb > kPooledQkMaxBlocks) return SPARSED_ERR_UNSUPPORTED;
  if ((st = prepare_pattern(out, shape->batch, shape->heads_q, nb, params->block_size, k_pre + k_gen)) != SPARSED_OK)
    return st;
  size_t need = 0;
  if ((st = sparsed_workspace_bytes(SPARSED_OP_SELECT_POOLED_QK, shape, params, &need)) != SPARSED_OK) return st;
  if ((st = check_ws(ws, ws_bytes, need)) != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  PooledQkParams p;
  p.q = q;
  p.k = k;
  p.q_stride_b = rs.q[0];
  p.q_stride_h = rs.q[1];
  p.q_stride_t = rs.q[2];
  p.k_stride_b = rs.k[0];
  p.k_stride_h = rs.k[1];
  p.k_stride_t = rs.k[2];
  p.means = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + SPARSED_STATUS_BYTES);
  p.scores = scores_out_or_null;
  p.row_ptr = out->row_ptr;
  p.col_idx = out->col_idx;
  p.batch = shape->batch;
  p.heads_q = shape->heads_q;
  p.group = shape->heads_q / shape->heads_kv;
  p.nb = nb;
  p.block_size = params->block_size;
  p.pb = pb;
  p.k_pre = k_pre;
  p.k_gen = k_gen;
  p.scale_log2 = rs.scale_log2;
  cudaError_t e = launch_pooled_qk_select(p, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

sparsed_status sparsed_attn_sparse(const sparsed_shape* shape, const sparsed_pattern* pattern, const void* q,
                                   const void* k, const void* v, void* o, void* ws, size_t ws_bytes,
                                   void* cuda_stream) {
  Resolved rs;
  sparsed_status st = check_shape(shape, true, &rs);
  if (st != SPARSED_OK) return st;
  if (q == nullptr || k == nullptr || v == nullptr || o == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return SPARSED_ERR_ALIGNMENT;
  if (pattern == nullptr || pattern->row_ptr == nullptr || pattern->col_idx == nullptr) return SPARSED_ERR_PATTERN;
  if (!aligned4(pattern->row_ptr) || !aligned4(pattern->col_idx)) return SPARSED_ERR_ALIGNMENT;
  if (pattern->block_size != 32 && pattern->block_size != 64 && pattern->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (pattern->batch != shape->batch || pattern->heads_q != shape->heads_q || pattern->num_blocks < 1 ||
      static_cast<int64_t>(pattern->num_blocks) * pattern->block_size != shape->seq_len)
    return SPARSED_ERR_PATTERN;
  if ((st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES)) != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  const int bs = pattern->block_size;
  if (pattern->num_blocks > attn_sparse_max_blocks(bs)) return SPARSED_ERR_UNSUPPORTED;
  CUtensorMap tq, tk, tv, to;
  if ((st = make_tensor_map(&tq, q, shape->batch, shape->heads_q, shape->seq_len, rs.q, 128)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&to, o, shape->batch, shape->heads_q, shape->seq_len, rs.o, 128)) != SPARSED_OK) return st;
  const int kv_box = bs < 64 ? bs : 64;
  if ((st = make_tensor_map(&tk, k, shape->batch, shape->heads_kv, shape->seq_len, rs.k, kv_box)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&tv, v, shape->batch, shape->heads_kv, shape->seq_len, rs.v, kv_box)) != SPARSED_OK) return st;
  AttnParams p;
  p.o = o;
  p.o_stride_b = rs.o[0];
  p.o_stride_h = rs.o[1];
  p.o_stride_t = rs.o[2];
  p.lse = nullptr;
  p.tile_lse = nullptr;
  p.stat_keys = 64;
  p.slow_path_events = reinterpret_cast<unsigned long long*>(static_cast<uint8_t*>(ws) + 32);
  p.seq_len = shape->seq_len;
  p.heads_q = shape->heads_q;
  p.group = shape->heads_q / shape->heads_kv;
  p.num_q_tiles = (shape->seq_len + 127) / 128;
  p.num_blocks = pattern->num_blocks;
  p.num_items = shape->batch * shape->heads_q * p.num_q_tiles;
  // block lists: as many CTAs as are resident at once, each running through its share of the query tiles, so
  // that only a CTA's first tile pays the start-up chain (+16 % at 4 blocks per row, +5 % at 14, +1 % at 52)
  p.max_ctas = attn_max_ctas();
  p.scale_log2 = rs.scale_log2;
  p.row_ptr = pattern->row_ptr;
  p.col_idx = pattern->col_idx;
  p.col_capacity = pattern->col_capacity;
  p.status = static_cast<DeviceStatus*>(ws);
  cudaError_t e = launch_attn_sparse(tq, tk, tv, to, p, shape->batch, bs, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

sparsed_status sparsed_select_from_scores(const sparsed_select_params* params, const float* scores, int32_t batch,
                                          int32_t heads_q, int32_t num_blocks, sparsed_pattern* out, void* ws,
                                          size_t ws_bytes, void* cuda_stream) {
  if (scores == nullptr || batch < 1 || heads_q < 1 || num_blocks < 1) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(scores)) return SPARSED_ERR_ALIGNMENT;
  int pb = 0, k_pre = 0, k_gen = 0;
  sparsed_status st = kept_counts(params, num_blocks, &pb, &k_pre, &k_gen);
  if (st != SPARSED_OK) return st;
  if ((st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES)) != SPARSED_OK) return st;
  if (out == nullptr || out->row_ptr == nullptr || out->col_idx == nullptr) return SPARSED_ERR_PATTERN;
  if ((st = check_arch()) != SPARSED_OK) return st;
  return run_topk(scores, batch, heads_q, num_blocks, params->block_size, pb, k_pre, k_gen, out,
                  static_cast<cudaStream_t>(cuda_stream));
}

sparsed_status sparsed_select_pattern(const sparsed_shape* shape, const sparsed_select_params* params, const void* q,
                                      const void* k, const float* lse_or_null, sparsed_pattern* out,
                                      float* scores_out_or_null, void* ws, size_t ws_bytes, void* cuda_stream) {
  Resolved rs;
  sparsed_status st = check_shape(shape, false, &rs);
  if (st != SPARSED_OK) return st;
  if (params == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (params->block_size != 32 && params->block_size != 64 && params->block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (shape->seq_len % params->block_size != 0) return SPARSED_ERR_ALIGNMENT;
  const int nb = shape->seq_len / params->block_size;
  int pb = 0, k_pre = 0, k_gen = 0;
  if ((st = kept_counts(params, nb, &pb, &k_pre, &k_gen)) != SPARSED_OK) return st;
  if (q == nullptr || k == nullptr) return SPARSED_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(lse_or_null) || !aligned16(scores_out_or_null))
    return SPARSED_ERR_ALIGNMENT;
  if ((st = prepare_pattern(out, shape->batch, shape->heads_q, nb, params->block_size, k_pre + k_gen)) != SPARSED_OK)
    return st;
  // With few enough blocks per row the pooled-scoring kernel ranks each block-row in its own
  // tail; A' then goes to memory only if the caller asked for it.
  const bool fused = nb <= kFusedTopkMaxBlocks && params->block_size != 32;
  const size_t bh = static_cast<size_t>(shape->batch) * shape->heads_q;
  const size_t score_bytes = round_up(bh * nb * nb * 4, 256);
  const size_t lse_bytes = round_up(bh * static_cast<size_t>(shape->seq_len) * 4, 256);
  const bool need_score_ws = !fused && scores_out_or_null == nullptr;
  const size_t required = SPARSED_STATUS_BYTES + (need_score_ws ? score_bytes : 0) + (lse_or_null ? 0 : lse_bytes);
  if ((st = check_ws(ws, ws_bytes, required)) != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* scores = scores_out_or_null;
  size_t off = SPARSED_STATUS_BYTES;
  if (need_score_ws) {
    scores = reinterpret_cast<float*>(base + off);
    off += score_bytes;
  }
  CUtensorMap tq, tk;
  if ((st = make_tensor_map(&tq, q, shape->batch, shape->heads_q, shape->seq_len, rs.q, 128)) != SPARSED_OK) return st;
  if ((st = make_tensor_map(&tk, k, shape->batch, shape->heads_kv, shape->seq_len, rs.k, 128)) != SPARSED_OK) return st;
  ScoreParams sp;
  sp.scores = scores;
  sp.lse = lse_or_null;
  sp.seq_len = shape->seq_len;
  sp.heads_q = shape->heads_q;
  sp.group = shape->heads_q / shape->heads_kv;
  sp.block_size = params->block_size;
  sp.scale_log2 = rs.scale_log2;
  sp.status = static_cast<DeviceStatus*>(ws);
  sp.row_ptr = fused ? out->row_ptr : nullptr;
  sp.col_idx = fused ? out->col_idx : nullptr;
  sp.pb = pb;
  sp.k_pre = k_pre;
  sp.k_gen = k_gen;
  if (lse_or_null == nullptr) {
    float* lse_buf = reinterpret_cast<float*>(base + off);
    cudaError_t e = launch_row_stats(tq, tk, sp, lse_buf, shape->batch, stream);
    if (e != cudaSuccess) return cuda_fail(e);
    sp.lse = lse_buf;
  }
  cudaError_t e = launch_pooled_scores(tq, tk, sp, shape->batch, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  if (fused) return SPARSED_OK;
  return run_topk(scores, shape->batch, shape->heads_q, nb, params->block_size, pb, k_pre, k_gen, out, stream);
}

sparsed_status sparsed_attention_step(const sparsed_shape* shape, const sparsed_select_params* params,
                                      int32_t step_1based, int32_t total_steps, double skip, const void* q,
                                      const void* k, const void* v, void* o, sparsed_pattern* pattern, void* ws,
                                      size_t ws_bytes, void* cuda_stream, int32_t* mode_out_or_null) {
  const int32_t mode = sparsed_schedule_mode(step_1based, total_steps, skip);
  if (mode < 0) return SPARSED_ERR_INVALID_ARG;
  if (mode_out_or_null != nullptr) *mode_out_or_null = mode;
  if (mode == SPARSED_MODE_FULL) return sparsed_attn_full(shape, q, k, v, o, nullptr, ws, ws_bytes, cuda_stream);
  if (mode == SPARSED_MODE_SPARSE) return sparsed_attn_sparse(shape, pattern, q, k, v, o, ws, ws_bytes, cuda_stream);
  // the switch step
  if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
  size_t need = 0;
  sparsed_status st = sparsed_workspace_bytes(SPARSED_OP_ATTENTION_STEP, shape, params, &need);
  if (st != SPARSED_OK) return st;
  if ((st = check_ws(ws, ws_bytes, need)) != SPARSED_OK) return st;
  const size_t bh = static_cast<size_t>(shape->batch) * shape->heads_q;
  const size_t lse_bytes = round_up(bh * static_cast<size_t>(shape->seq_len) * 4, 256);
  uint8_t* base = static_cast<uint8_t*>(ws);
  if (step_uses_stats(shape, params)) {
    float* lse = reinterpret_cast<float*>(base + SPARSED_STATUS_BYTES);
    float* stats = reinterpret_cast<float*>(base + SPARSED_STATUS_BYTES + lse_bytes);
    if ((st = sparsed_attn_full_stats(shape, params->block_size, q, k, v, o, lse, stats, ws, ws_bytes, cuda_stream)) != SPARSED_OK)
      return st;
    return sparsed_select_from_stats(shape, params, lse, stats, pattern, nullptr, ws, ws_bytes, cuda_stream);
  }
  // [status][A' scratch of sparsed_select_pattern][LSE of the full pass]
  const size_t nb = static_cast<size_t>(shape->seq_len / params->block_size);
  const size_t score_bytes = round_up(bh * nb * nb * 4, 256);
  float* lse = reinterpret_cast<float*>(base + SPARSED_STATUS_BYTES + score_bytes);
  if ((st = sparsed_attn_full(shape, q, k, v, o, lse, ws, ws_bytes, cuda_stream)) != SPARSED_OK) return st;
  return sparsed_select_pattern(shape, params, q, k, lse, pattern, nullptr, ws, SPARSED_STATUS_BYTES + score_bytes,
                                cuda_stream);
}

sparsed_status sparsed_attention_step_variant(const sparsed_shape* shape, const sparsed_select_params* params,
                                              int32_t variant, int32_t step_1based, int32_t total_steps, double skip,
                                              const void* q, const void* k, const void* v, void* o,
                                              sparsed_pattern* pattern, void* ws, size_t ws_bytes, void* cuda_stream,
                                              int32_t* mode_out_or_null) {
  if (params == nullptr) return SPARSED_ERR_INVALID_ARG;
  if ((variant & ~(SPARSED_VARIANT_NO_REUSE | SPARSED_VARIANT_NO_ISOLATION)) != 0) return SPARSED_ERR_INVALID_ARG;
  sparsed_select_params p2 = *params;
  if (variant & SPARSED_VARIANT_NO_ISOLATION) p2.prefill_len = 0;
  const int32_t mode = sparsed_schedule_mode(step_1based, total_steps, skip);
  if (mode < 0) return SPARSED_ERR_INVALID_ARG;
  if (mode == SPARSED_MODE_SPARSE && (variant & SPARSED_VARIANT_NO_REUSE)) {
    // "without Sparse Reusing": this step's own Q and K give this step's pattern (row statistics
    // pass + pooled scoring + ranking), then the block-sparse attention runs on it
    if (mode_out_or_null != nullptr) *mode_out_or_null = mode;
    sparsed_status st = sparsed_select_pattern(shape, &p2, q, k, nullptr, pattern, nullptr, ws, ws_bytes, cuda_stream);
    if (st != SPARSED_OK) return st;
    return sparsed_attn_sparse(shape, pattern, q, k, v, o, ws, ws_bytes, cuda_stream);
  }
  return sparsed_attention_step(shape, &p2, step_1based, total_steps, skip, q, k, v, o, pattern, ws, ws_bytes,
                                cuda_stream, mode_out_or_null);
}

sparsed_status sparsed_build_window_pattern(int32_t batch, int32_t heads_q, int32_t num_blocks, int32_t block_size,
                                            int32_t sink_blocks, int32_t window_blocks, sparsed_pattern* out,
                                            void* cuda_stream) {
  if (batch < 1 || heads_q < 1 || num_blocks < 1 || sink_blocks < 0 || window_blocks < 1) return SPARSED_ERR_INVALID_ARG;
  if (block_size != 32 && block_size != 64 && block_size != 128) return SPARSED_ERR_UNSUPPORTED;
  if (num_blocks > 16384) return SPARSED_ERR_UNSUPPORTED;
  if (out == nullptr || out->row_ptr == nullptr || out->col_idx == nullptr) return SPARSED_ERR_PATTERN;
  if (!aligned4(out->row_ptr) || !aligned4(out->col_idx)) return SPARSED_ERR_ALIGNMENT;
  const int sink = sink_blocks < num_blocks ? sink_blocks : num_blocks;
  const int half = (window_blocks - 1) / 2;
  const int64_t per_head = window_pattern_nnz_per_head(num_blocks, sink, half);
  const int64_t bh = static_cast<int64_t>(batch) * heads_q;
  const int64_t nnz = per_head * bh;
  if (nnz >= INT32_MAX || bh * num_blocks >= INT32_MAX) return SPARSED_ERR_UNSUPPORTED;
  if (out->col_capacity < nnz) return SPARSED_ERR_PATTERN;
  cudaError_t e = launch_window_pattern(out->row_ptr, out->col_idx, static_cast<int>(bh), num_blocks, sink, half,
                                        static_cast<int>(per_head), static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(e);
  out->nnz = nnz;
  out->block_size = block_size;
  out->num_blocks = num_blocks;
  out->batch = batch;
  out->heads_q = heads_q;
  return SPARSED_OK;
}

sparsed_status sparsed_pattern_validate(const sparsed_pattern* pattern, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (pattern == nullptr || pattern->row_ptr == nullptr || pattern->col_idx == nullptr) return SPARSED_ERR_PATTERN;
  if (pattern->batch < 1 || pattern->heads_q < 1 || pattern->num_blocks < 1) return SPARSED_ERR_PATTERN;
  if (!aligned4(pattern->row_ptr) || !aligned4(pattern->col_idx)) return SPARSED_ERR_ALIGNMENT;
  sparsed_status st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES);
  if (st != SPARSED_OK) return st;
  const int64_t rows = static_cast<int64_t>(pattern->batch) * pattern->heads_q * pattern->num_blocks;
  if (rows >= INT32_MAX) return SPARSED_ERR_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* flag = reinterpret_cast<int*>(static_cast<uint8_t*>(ws) + 16);
  cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), stream);
  if (e != cudaSuccess) return cuda_fail(e);
  e = launch_pattern_validate(pattern->row_ptr, pattern->col_idx, static_cast<int>(rows), pattern->num_blocks,
                              pattern->col_capacity, flag, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  int host_flag = 0;
  e = cudaMemcpyAsync(&host_flag, flag, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return host_flag == 0 ? SPARSED_OK : SPARSED_ERR_PATTERN;
}

sparsed_status sparsed_selftest_wait_timeout(void* ws, size_t ws_bytes, void* cuda_stream) {
  sparsed_status st = check_ws(ws, ws_bytes, SPARSED_STATUS_BYTES);
  if (st != SPARSED_OK) return st;
  if ((st = check_arch()) != SPARSED_OK) return st;
  cudaError_t e = launch_wait_timeout_selftest(static_cast<DeviceStatus*>(ws), 99, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? SPARSED_OK : cuda_fail(e);
}

sparsed_status sparsed_last_device_status(void* ws, void* cuda_stream, int32_t* code, int32_t* where) {
  if (ws == nullptr) return SPARSED_ERR_WORKSPACE;
  if (!aligned4(ws)) return SPARSED_ERR_ALIGNMENT;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int32_t host[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e);
  if (code != nullptr) *code = host[0];
  if (where != nullptr) *where = host[1];
  return host[0] == 0 ? SPARSED_OK : SPARSED_ERR_DEVICE_TIMEOUT;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Selection without a caller workspace: the scratch lives in this library's device image.
// ------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = SPARSED_STATIC_SCRATCH_BYTES;

// Scratch for sparsed_select_pattern_static: status block, pooled scores A', and the LSE
// rows when the caller has none. One copy per GPU that loads the library, held until exit.
static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

std::mutex g_scratch_mutex;
void* g_scratch_addr[64] = {};

// In host code `g_select_scratch` is only a handle for the runtime, not a device address:
// the address a kernel may use is looked up once per device with that device current.
sparsed_status static_scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return SPARSED_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_select_scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    if (ptr == nullptr) return cuda_fail(cudaErrorInvalidSymbol);
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return SPARSED_OK;
}

}  // namespace

extern "C" sparsed_status sparsed_select_pattern_static(const sparsed_shape* shape,
                                                        const sparsed_select_params* params, const void* q,
                                                        const void* k, const float* lse_or_null,
                                                        sparsed_pattern* out, void* cuda_stream) {
  if (shape == nullptr || params == nullptr) return SPARSED_ERR_INVALID_ARG;
  // Size check first, on the host, so that an oversized request never reaches the device.
  size_t full = 0;
  sparsed_status st = sparsed_workspace_bytes(SPARSED_OP_SELECT_PATTERN, shape, params, &full);
  if (st != SPARSED_OK) return st;
  const size_t bh = static_cast<size_t>(shape->batch) * static_cast<size_t>(shape->heads_q);
  const size_t lse_bytes = round_up(bh * static_cast<size_t>(shape->seq_len) * 4, 256);
  const size_t needed = full - (lse_or_null != nullptr ? lse_bytes : 0);
  if (needed > kStaticScratchBytes) return SPARSED_ERR_WORKSPACE;
  void* scratch = nullptr;
  if ((st = static_scratch_address(&scratch)) != SPARSED_OK) return st;
  // The array keeps whatever the previous call left: the status block must start at zero;
  // scores and LSE rows are fully rewritten by the kernels before anything reads them.
  cudaError_t e = cudaMemsetAsync(scratch, 0, SPARSED_STATUS_BYTES, static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(e);
  return sparsed_select_pattern(shape, params, q, k, lse_or_null, out, nullptr, scratch, kStaticScratchBytes,
                                cuda_stream);
}

