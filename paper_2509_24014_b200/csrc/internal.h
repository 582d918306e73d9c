// Internal host-side interfaces between the C ABI layer and the kernel launchers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "sm100_primitives.cuh"

namespace sparsed {

// Per-kernel record of the dynamic shared-memory limit already granted on each device, so that
// cudaFuncSetAttribute runs once per (kernel, device) instead of on every launch. Safe to use from
// several host threads: the fast path is one atomic load, the slow path is serialised.
struct SmemLimit {
  std::atomic<int> granted[64];
  std::mutex slow;
};

template <class Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, SmemLimit& lim) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && lim.granted[dev].load(std::memory_order_acquire) >= bytes) return cudaSuccess;
  std::lock_guard<std::mutex> lock(lim.slow);
  if (tracked && lim.granted[dev].load(std::memory_order_relaxed) >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && tracked) lim.granted[dev].store(bytes, std::memory_order_release);
  return e;
}

// Parameters shared by the dense and the block-sparse attention kernels.
struct AttnParams {
  void* o;                 // bf16 [B,Hq,L,D]; used by the plain dense kernel, which stores rows itself (the others
                           // write O through its tensor map)
  int64_t o_stride_b, o_stride_h, o_stride_t;
  float* lse;              // fp32 [B,Hq,L] or null
  float* tile_lse;         // fp32 [B*Hq, ceil(L/128), ceil(L/stat_keys), 128] or null: base-2 log-sum-exp of each row over each group of stat_keys keys
  int stat_keys;           // 32, 64 or 128
  unsigned long long* slow_path_events;  // counts warp-level rescales of the output accumulator, or null
  int seq_len;
  int heads_q;
  int group;               // heads_q / heads_kv
  int num_q_tiles;         // 128-row query tiles per (batch, head)
  int num_blocks;          // sparse only: pattern blocks per row (seq_len / block_size)
  int num_items;           // batch * heads_q * num_q_tiles: 128-row query tiles in all
  int max_ctas;            // > 0: launch at most this many CTAs and let each run through several items
  float scale_log2;        // softmax scale * log2(e)
  const int32_t* row_ptr;  // sparse only
  const int32_t* col_idx;  // sparse only
  int64_t col_capacity;    // sparse only: entries of col_idx that may be read
  DeviceStatus* status;
};

// Parameters of the pooled-scoring kernel.
struct ScoreParams {
  float* scores;           // fp32 [B,Hq,nb,nb], or null when only the pattern is wanted (fused top-k)
  const float* lse;        // fp32 [B,Hq,L], natural log
  int seq_len;
  int heads_q;
  int group;
  int block_size;          // 32, 64 or 128
  float scale_log2;
  DeviceStatus* status;
  // fused selection (row_ptr != null): each CTA ranks the block-row(s) it has just pooled
  int32_t* row_ptr;
  int32_t* col_idx;
  int pb, k_pre, k_gen;
};

// Largest number of key blocks per row the pooled-scoring kernel can rank in its own tail.
constexpr int kFusedTopkMaxBlocks = 1024;

// Parameters of the kernel that pools per-tile row statistics into A' and ranks it.
struct PoolParams {
  const float* tile_lse;   // fp32 [B*Hq, ceil(L/128), L/block_size, 128], base-2
  const float* lse;        // fp32 [B,Hq,L], natural log
  float* scores;           // fp32 [B,Hq,nb,nb] or null
  int32_t* row_ptr;
  int32_t* col_idx;
  int seq_len;
  int block_size;          // 32, 64 or 128 (= keys per statistic)
  int pb, k_pre, k_gen;
  int bh;                  // B * Hq
};

struct TopkParams {
  const float* scores;     // fp32 [rows, nb]
  int32_t* row_ptr;
  int32_t* col_idx;
  int rows;                // B * Hq * nb
  int nb;
  int pb;                  // prefill blocks
  int k_pre, k_gen;
};

// Parameters of the block-mean estimate of A' (not the paper's scorer) and the selection from it.
struct PooledQkParams {
  const void* q;           // bf16 [B,Hq,L,128]
  const void* k;           // bf16 [B,Hkv,L,128]
  int64_t q_stride_b, q_stride_h, q_stride_t;
  int64_t k_stride_b, k_stride_h, k_stride_t;
  float* means;            // fp32 scratch: [B,Hq,nb,128] then [B,Hkv,nb,128]
  float* scores;           // fp32 [B,Hq,nb,nb] or null
  int32_t* row_ptr;
  int32_t* col_idx;
  int batch, heads_q, group;
  int nb, block_size;
  int pb, k_pre, k_gen;
  float scale_log2;
};

// Largest number of key blocks per row the block-mean selection kernel holds in shared memory.
constexpr int kPooledQkMaxBlocks = 1024;

size_t pooled_qk_means_bytes(int batch, int heads_q, int heads_kv, int nb);
cudaError_t launch_pooled_qk_select(const PooledQkParams& p, cudaStream_t stream);
// (`to`: tensor map of the output, boxes of 64 x 128 rows like Q's; the kernels write O through it)
cudaError_t launch_attn_dense(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                              const CUtensorMap& to, const AttnParams& p, int batch, cudaStream_t stream);
// The same pass with the MMAs spanning CTA pairs (cta_group::2); K tensor map with 32-row boxes.
cudaError_t launch_attn_dense_pair(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                   const CUtensorMap& to, const AttnParams& p, cudaStream_t stream);
int attn_sparse_max_blocks(int block_size);   // most key blocks per row the sparse kernel handles
cudaError_t launch_attn_sparse(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const CUtensorMap& to, const AttnParams& p, int batch, int block_size,
                               cudaStream_t stream);
cudaError_t launch_row_stats(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, float* lse_out,
                             int batch, cudaStream_t stream);
cudaError_t launch_pooled_scores(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, int batch,
                                 cudaStream_t stream);
cudaError_t launch_topk_csr(const TopkParams& p, cudaStream_t stream);
int pool_select_max_blocks();   // most key blocks per row the statistics path handles
cudaError_t launch_pool_select(const PoolParams& p, cudaStream_t stream);
int64_t window_pattern_nnz_per_head(int nb, int sink, int half);
cudaError_t launch_window_pattern(int32_t* row_ptr, int32_t* col_idx, int bh, int nb, int sink, int half,
                                  int per_head_nnz, cudaStream_t stream);
cudaError_t launch_wait_timeout_selftest(DeviceStatus* status, int where, cudaStream_t stream);
cudaError_t launch_pattern_validate(const int32_t* row_ptr, const int32_t* col_idx, int rows, int nb,
                                    int64_t capacity, int* bad_flag, cudaStream_t stream);

}  // namespace sparsed
