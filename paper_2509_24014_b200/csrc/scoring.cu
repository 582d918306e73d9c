// Block-pooled attention scores A' = avgpool(softmax(Q K^T / sqrt(d)), block_size)
// ("Isolated Selection"; the avgpool line of Algorithm 1), streamed one 128-row query tile
// at a time so that the l x l matrix is never stored.
//
// Two kernels built from one template:
//   * row statistics : LSE_i = ln sum_j exp(s_ij) by online max/sum (only needed when the
//                      caller has no LSE from the full-attention pass of the same step);
//   * pooled scores  : p_ij = exp(s_ij - LSE_i) is the exactly normalised probability, so
//                      each 128x128 logit tile can be reduced to its block sums at once.
// Pipeline per CTA: warp 4 streams K tiles by TMA (two stages), warp 5 issues S = Q K^T
// into one of two tensor-memory buffers, warps 0-3 (one thread per query row) exponentiate
// and reduce. Sums run in a fixed order, so results are bitwise reproducible.
// With a pattern to fill (row_ptr != null) warp 0 also keeps the block-row(s) it produced as
// ordered keys in shared memory and, after the last tile, runs the isolated top-k of Eq. 5/6
// on them and writes the CSR lists: selection then needs no pass over A' in memory.
#include "internal.h"
#include "topk_device.cuh"

namespace sparsed {
namespace {

constexpr int kHeadDim = 128;
constexpr int kTile = 128;
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;
constexpr int kStages = 2;

struct ScoreSmem {
  alignas(1024) __nv_bfloat16 q[2][kTile * 64];
  alignas(1024) __nv_bfloat16 k[kStages][2][kTile * 64];
  uint64_t q_full, k_full[kStages], s_full[2], s_empty[2], partial_full[4];
  float partial[4][4][2];  // [tile % 4][warp][column half]
  uint32_t keys[2][kFusedTopkMaxBlocks];  // ordered keys of the block-row(s) of this CTA (fused top-k)
  int hist[256];
  uint32_t tmem_base;
  int abort_flag;
};

template <bool kStatsOnly>
__global__ void __launch_bounds__(kThreads, 2)
score_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
             const ScoreParams p, float* lse_out) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0u) {
    if (threadIdx.x == 0 && atomicCAS(&p.status->code, 0, 2) == 0) p.status->where = 2;
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const int num_q_tiles = (p.seq_len + kTile - 1) / kTile;
  const int num_tiles = num_q_tiles;
  const int q_tile = blockIdx.x % num_q_tiles;
  const int bh = blockIdx.x / num_q_tiles;
  const int head = bh % p.heads_q;
  const int batch = bh / p.heads_q;
  const int kv_head = head / p.group;
  const int q_row0 = q_tile * kTile;

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    static_assert(kStages == 2, "K stage and S buffer of a tile share one index and one completion barrier");
    for (int s = 0; s < kStages; ++s) mbar_init(&sm.k_full[s], 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.s_full[s], 1);
      mbar_init(&sm.s_empty[s], 128);
    }
    for (int s = 0; s < 4; ++s) mbar_init(&sm.partial_full[s], 4);
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 5) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 4) {
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      mbar_expect_tx(&sm.q_full, kTile * kHeadDim * 2);
      tma_load_4d(sm.q[0], &tm_q, &sm.q_full, 0, q_row0, head, batch);
      tma_load_4d(sm.q[1], &tm_q, &sm.q_full, 64, q_row0, head, batch);
      for (int it = 0; it < num_tiles; ++it) {
        const int s = it % kStages;
        const int use = it / kStages;
        // the stage's previous K tile has been read once the S buffer of the same index is complete
        if (use > 0 && !mbar_wait(&sm.s_full[s], (use - 1) & 1, &sm.abort_flag, p.status, 40)) break;
        mbar_expect_tx(&sm.k_full[s], kTile * kHeadDim * 2);
        tma_load_4d(sm.k[s][0], &tm_k, &sm.k_full[s], 0, it * kTile, kv_head, batch);
        tma_load_4d(sm.k[s][1], &tm_k, &sm.k_full[s], 64, it * kTile, kv_head, batch);
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTile, kTile, false, false);
      const uint32_t q_addr[2] = {smem_u32(sm.q[0]), smem_u32(sm.q[1])};
      bool ok = mbar_wait(&sm.q_full, 0, &sm.abort_flag, p.status, 50);
      for (int it = 0; ok && it < num_tiles; ++it) {
        const int s = it % kStages;
        const int buf = it & 1;
        if (!mbar_wait(&sm.k_full[s], (it / kStages) & 1, &sm.abort_flag, p.status, 51)) break;
        if (it >= 2 && !mbar_wait(&sm.s_empty[buf], ((it >> 1) - 1) & 1, &sm.abort_flag, p.status, 52)) break;
        tc_fence_after();
        const uint32_t k_addr[2] = {smem_u32(sm.k[s][0]), smem_u32(sm.k[s][1])};
#pragma unroll
        for (int kk = 0; kk < kHeadDim / 16; ++kk) {
          const uint32_t off = (kk & 3) * 32;
          umma_ss(tmem + buf * kTile, umma_smem_desc_sw128(q_addr[kk >> 2] + off, 16, 1024),
                  umma_smem_desc_sw128(k_addr[kk >> 2] + off, 16, 1024), idesc, kk > 0);
        }
        umma_commit(&sm.s_full[buf]);   // one commit: "S ready" for the softmax warps, "K stage free" for the producer
      }
    }
  } else {
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const float scale_log2 = p.scale_log2;
    const int row = q_row0 + tid;
    const bool row_valid = row < p.seq_len;
    // pooled mode: natural-log LSE -> base-2 offset
    float lse2 = 0.f;
    if constexpr (!kStatsOnly) {
      lse2 = row_valid ? p.lse[static_cast<int64_t>(bh) * p.seq_len + row] * 1.44269504088896341f : INFINITY;
    }
    float m_run = -INFINITY, l_run = 0.f;
    const int nb = p.seq_len / p.block_size;
    const bool half_blocks = (p.block_size == 64);
    const float inv_area = 1.f / (static_cast<float>(p.block_size) * static_cast<float>(p.block_size));
    const bool fuse_topk = (!kStatsOnly) && (p.row_ptr != nullptr);
    bool ok = true;
    for (int it = 0; it < num_tiles; ++it) {
      const int buf = it & 1;
      if (!mbar_wait(&sm.s_full[buf], (it >> 1) & 1, &sm.abort_flag, p.status, 60)) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t tS = tmem + buf * kTile + lane_base;
      const int valid_cols = min(kTile, p.seq_len - it * kTile);
      if constexpr (kStatsOnly) {
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < kTile / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tS + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j < valid_cols) mx = fmaxf(mx, __uint_as_float(r[j]));
        }
        const float m_new = fmaxf(m_run, mx * scale_log2);
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < kTile / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tS + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float e = fast_exp2(fmaf(__uint_as_float(r[j]), scale_log2, -m_new));
            sum += (c * 32 + j < valid_cols) ? e : 0.f;
          }
        }
        l_run = l_run * fast_exp2(m_run - m_new) + sum;
        m_run = m_new;
        tc_fence_before();
        mbar_arrive(&sm.s_empty[buf]);
      } else {
        float half_sum[2] = {0.f, 0.f};
        float quarter[4];
#pragma unroll
        for (int c = 0; c < kTile / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tS + c * 32, r);
          tmem_wait_ld();
          float acc = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            acc += fast_exp2(fmaf(__uint_as_float(r[j]), scale_log2, -lse2));
          half_sum[c >> 1] += acc;
          quarter[c] = acc;
        }
        if (p.block_size == 32) {
          // 32-key blocks: a warp's 32 rows are one query block and each 32-column chunk one key
          // block, so every warp finishes its own four scores (scores always go to memory here)
          tc_fence_before();
          mbar_arrive(&sm.s_empty[buf]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) quarter[c] += __shfl_xor_sync(0xffffffffu, quarter[c], off);
          }
          const int ib = q_tile * 4 + warp;
          if (lane < 4 && ib < nb) {
            const int jb = it * 4 + lane;
            const float total = lane == 0 ? quarter[0] : (lane == 1 ? quarter[1] : (lane == 2 ? quarter[2] : quarter[3]));
            if (jb < nb) p.scores[(static_cast<int64_t>(bh) * nb + ib) * nb + jb] = total * inv_area;
          }
          continue;
        }
        tc_fence_before();
        mbar_arrive(&sm.s_empty[buf]);
        // reduce over the 32 rows of this warp (fixed butterfly order)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          half_sum[0] += __shfl_xor_sync(0xffffffffu, half_sum[0], off);
          half_sum[1] += __shfl_xor_sync(0xffffffffu, half_sum[1], off);
        }
        // Per-warp partial sums go through a 4-deep ring in shared memory; the S buffers keep
        // every warp within two tiles of the others, so a slot is never rewritten while read.
        const int slot = it & 3;
        if (lane == 0) {
          sm.partial[slot][warp][0] = half_sum[0];
          sm.partial[slot][warp][1] = half_sum[1];
          mbar_arrive(&sm.partial_full[slot]);
        }
        if (warp == 0 && lane < 4) {
          if (!mbar_wait(&sm.partial_full[slot], (it >> 2) & 1, &sm.abort_flag, p.status, 61)) {
            ok = false;
          } else if (!half_blocks) {
            if (lane == 0) {
              const float* pp = &sm.partial[slot][0][0];
              const float total = ((pp[0] + pp[1]) + (pp[2] + pp[3])) + ((pp[4] + pp[5]) + (pp[6] + pp[7]));
              const float score = total * inv_area;
              if (p.scores != nullptr) p.scores[(static_cast<int64_t>(bh) * nb + q_tile) * nb + it] = score;
              if (fuse_topk) sm.keys[0][it] = ordered_key(score);
            }
          } else {
            const int rh = lane >> 1, ch = lane & 1;  // row half (warps 2rh, 2rh+1), column half
            const int ib = q_tile * 2 + rh, jb = it * 2 + ch;
            if (ib < nb && jb < nb) {
              const float total = sm.partial[slot][2 * rh][ch] + sm.partial[slot][2 * rh + 1][ch];
              const float score = total * inv_area;
              if (p.scores != nullptr) p.scores[(static_cast<int64_t>(bh) * nb + ib) * nb + jb] = score;
              if (fuse_topk) sm.keys[rh][jb] = ordered_key(score);
            }
          }
        }
        __syncwarp();
      }
    }
    if constexpr (!kStatsOnly) {
      if (fuse_topk && warp == 0) {
        // warp 0 wrote every key of this CTA's block-row(s); rank them now (Eq. 5 / Eq. 6)
        const bool all_ok = __all_sync(0xffffffffu, ok);
        __syncwarp();
        if (all_ok) {
          const int k_total = p.k_pre + p.k_gen;
          const int rows_here = half_blocks ? 2 : 1;
          for (int rh = 0; rh < rows_here; ++rh) {
            const int ib = half_blocks ? q_tile * 2 + rh : q_tile;
            if (ib >= nb) break;
            const int64_t row = static_cast<int64_t>(bh) * nb + ib;
            warp_select_row(sm.keys[rh], nb, p.pb, p.k_pre, p.k_gen, sm.hist, p.col_idx + row * k_total, lane);
            if (lane == 0) {
              p.row_ptr[row] = static_cast<int32_t>(row * k_total);
              if (row == static_cast<int64_t>(gridDim.x / num_q_tiles) * nb - 1)
                p.row_ptr[row + 1] = static_cast<int32_t>((row + 1) * k_total);
            }
            __syncwarp();
          }
        }
      }
    }
    if constexpr (kStatsOnly) {
      if (ok && row_valid) lse_out[static_cast<int64_t>(bh) * p.seq_len + row] = (m_run + log2f(l_run)) * 0.69314718055994531f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <bool kStatsOnly>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, float* lse_out, int batch,
                   cudaStream_t stream) {
  auto kernel = score_kernel<kStatsOnly>;
  const int smem = static_cast<int>(sizeof(ScoreSmem));
  static SmemLimit limit;  // per template instantiation
  cudaError_t e = ensure_dynamic_smem(kernel, smem, limit);
  if (e != cudaSuccess) return e;
  const int num_q_tiles = (p.seq_len + kTile - 1) / kTile;
  const long long ctas = static_cast<long long>(batch) * p.heads_q * num_q_tiles;
  if (ctas <= 0) return cudaSuccess;
  kernel<<<static_cast<unsigned>(ctas), kThreads, smem, stream>>>(tq, tk, p, lse_out);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_row_stats(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, float* lse_out,
                             int batch, cudaStream_t stream) {
  return launch<true>(tq, tk, p, lse_out, batch, stream);
}

cudaError_t launch_pooled_scores(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, int batch,
                                 cudaStream_t stream) {
  return launch<false>(tq, tk, p, nullptr, batch, stream);
}

}  // namespace sparsed
