// Pattern selection from the row statistics of the switch step's full-attention pass
// ("Isolated Selection": A' = avgpool(A, block_size), then Eq. 5 / Eq. 6), without a second
// Q K^T pass.
//
// The dense attention kernel can record, for every query row i and every group g of block_size
// keys, v[g][i] = log2 sum_{j in g} 2^(s_ij), the group's share of the row's softmax denominator.
// With the row's final log-sum-exp, 2^(v[g][i] - LSE_i) is exactly the probability mass row i
// puts on key block g, so A'[ib][jb] is the sum of that mass over the rows of query block ib,
// divided by block_size^2.
//
// One CTA owns one 128-row query tile of one (batch, head), i.e. one, two or four query blocks.
// Statistics are read with 16-byte loads (four consecutive rows of one key block; the layout
// [bh][128-row query tile][key block][row] makes a CTA's reads one contiguous run), eight in flight
// per thread and six CTAs per SM (the best point of a sweep: 5.9 TB/s at 64k), exponentiated,
// parked in shared memory in chunks of 32 key blocks, and summed per key block and 32-row quarter
// in a fixed, bank-conflict-free order (bitwise reproducible); the next chunk's loads are issued
// before the current chunk is summed. The quarters are then combined into the CTA's block-row(s)
// of A', which are optionally written out, and one warp per block-row ranks it (warp_select_row)
// and writes the CSR list. HBM-bound: 4 * 128 * ceil(L/128) * (L / block_size) bytes read per
// (batch, head).
#include "internal.h"
#include "topk_device.cuh"

namespace sparsed {
namespace {

constexpr int kRows = 128;
#ifndef SPARSED_POOL_IN_FLIGHT
#define SPARSED_POOL_IN_FLIGHT 8
#endif
#ifndef SPARSED_POOL_CTAS_PER_SM
#define SPARSED_POOL_CTAS_PER_SM 6
#endif
constexpr int kInFlight = SPARSED_POOL_IN_FLIGHT;  // 16-byte loads each thread keeps in flight
constexpr int kChunk = 4 * kInFlight;  // tiles per transposition chunk: one batch of loads per thread
constexpr int kPitch = kRows + 4;   // floats per chunk row: keeps float4 stores aligned
constexpr int kMaxBlocks = 2048;    // key blocks per row: seq_len <= 2048 * block_size

// Shared memory (dynamic, sized for the actual sequence): the transposition chunk, the per-block
// mass of each 32-row quarter of the query tile, the ordered keys of this CTA's block-row(s), one
// top-k histogram per block-row.
struct PoolSmem {
  float* chunk;                     // [key block in chunk][kPitch]
  float* quarter_sum;               // [32-row quarter][key block]
  uint32_t* keys;                   // [block-row of this CTA][key block]
  int* hist;                        // [block-row][256]
};

__host__ __device__ inline size_t pool_smem_bytes(int nb, int rows_here) {
  return sizeof(float) * kChunk * kPitch + sizeof(float) * 4 * nb + sizeof(uint32_t) * rows_here * nb +
         sizeof(int) * 256 * rows_here;
}

__global__ void __launch_bounds__(kRows, SPARSED_POOL_CTAS_PER_SM) pool_select_kernel(const PoolParams p) {
  extern __shared__ __align__(16) uint8_t pool_smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = p.seq_len;
  const int bs = p.block_size;
  const int nb = L / bs;                    // key blocks per row = statistics per row
  const int rows_here = kRows / bs;         // block-rows of A' this CTA produces: 1, 2 or 4
  PoolSmem sm;
  {
    float* f = reinterpret_cast<float*>(pool_smem_raw);
    sm.chunk = f;
    f += kChunk * kPitch;
    sm.quarter_sum = f;
    f += 4 * nb;
    sm.keys = reinterpret_cast<uint32_t*>(f);
    sm.hist = reinterpret_cast<int*>(sm.keys + rows_here * nb);
  }
  const int num_q_tiles = (L + kRows - 1) / kRows;
  const int q_tile = blockIdx.x % num_q_tiles;
  const int bh = blockIdx.x / num_q_tiles;
  // Loading: lane l owns rows 4l..4l+3 of the query tile (one 16-byte load covers them), warp w
  // takes key blocks w, w+4, ... of the chunk. seq_len is a multiple of 32 here, so a group of four
  // rows is valid or invalid as a whole and 16-byte aligned.
  const int row4 = q_tile * kRows + lane * 4;
  const bool rows_valid = row4 < L;
  float4 lse2 = make_float4(INFINITY, INFINITY, INFINITY, INFINITY);
  if (rows_valid) {
    const float4 t = *reinterpret_cast<const float4*>(p.lse + static_cast<int64_t>(bh) * L + row4);
    const float c = 1.44269504088896341f;
    lse2 = make_float4(t.x * c, t.y * c, t.z * c, t.w * c);
  }
  // statistics layout [bh][query tile][key block][128 rows]: this CTA's share is one contiguous run
  const float* src = p.tile_lse + (static_cast<int64_t>(bh) * num_q_tiles + q_tile) * nb * kRows + lane * 4;

  // One batch = this thread's kInFlight loads of a chunk (warp w takes key blocks w, w+4, ... of it).
  // The next chunk's batch is issued before the current chunk is summed, so loads stay in flight
  // through the shared-memory phase.
  static_assert(kChunk == 4 * kInFlight, "one batch of loads per thread covers one chunk");
  static_assert(kChunk == 32, "the summation assigns one key block of the chunk to each lane");
  float4 v[kInFlight];
  auto issue = [&](int c0) {
    const int n_here = min(kChunk, nb - c0);
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int t = warp + 4 * u;
      v[u] = (rows_valid && t < n_here)
                 ? __ldcs(reinterpret_cast<const float4*>(src + static_cast<int64_t>(c0 + t) * kRows))
                 : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
  };
  issue(0);
  for (int c0 = 0; c0 < nb; c0 += kChunk) {
    const int n_here = min(kChunk, nb - c0);
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int t = warp + 4 * u;
      if (t < n_here) {
        const float4 e = make_float4(fast_exp2(v[u].x - lse2.x), fast_exp2(v[u].y - lse2.y),
                                     fast_exp2(v[u].z - lse2.z), fast_exp2(v[u].w - lse2.w));
        *reinterpret_cast<float4*>(sm.chunk + t * kPitch + lane * 4) = e;
      }
    }
    __syncthreads();
    if (c0 + kChunk < nb) issue(c0 + kChunk);
    {
      // Summing: warp w adds rows 32w..32w+31 (one quarter of the query tile), lane j key block j of
      // the chunk. Each lane starts at its own rotation of the 32 rows so that a warp's reads hit 32
      // different banks; the order is fixed per key block, so the result is reproducible.
      const int j = lane;
      if (j < n_here) {
        const float* rowp = sm.chunk + j * kPitch + warp * 32;
        float acc = 0.f;
#pragma unroll 8
        for (int r = 0; r < 32; ++r) acc += rowp[(r + 29 * j) & 31];
        sm.quarter_sum[warp * nb + c0 + j] = acc;
      }
    }
    __syncthreads();
  }

  const float inv_area = 1.f / (static_cast<float>(bs) * static_cast<float>(bs));
  for (int jb = tid; jb < nb; jb += kRows) {
    const float q0 = sm.quarter_sum[jb], q1 = sm.quarter_sum[nb + jb], q2 = sm.quarter_sum[2 * nb + jb],
                q3 = sm.quarter_sum[3 * nb + jb];
    float score[4];
    if (bs == 128) {
      score[0] = ((q0 + q1) + (q2 + q3)) * inv_area;
    } else if (bs == 64) {
      score[0] = (q0 + q1) * inv_area;
      score[1] = (q2 + q3) * inv_area;
    } else {
      score[0] = q0 * inv_area;
      score[1] = q1 * inv_area;
      score[2] = q2 * inv_area;
      score[3] = q3 * inv_area;
    }
#pragma unroll
    for (int rh = 0; rh < 4; ++rh) {
      const int ib = q_tile * rows_here + rh;
      if (rh < rows_here && ib < nb) {
        sm.keys[rh * nb + jb] = ordered_key(score[rh]);
        if (p.scores != nullptr) p.scores[(static_cast<int64_t>(bh) * nb + ib) * nb + jb] = score[rh];
      }
    }
  }
  __syncthreads();
  // one warp per block-row: isolated top-k (Eq. 5 / Eq. 6) and the CSR list
  if (warp < rows_here) {
    const int ib = q_tile * rows_here + warp;
    if (ib < nb) {
      const int k_total = p.k_pre + p.k_gen;
      const int64_t r = static_cast<int64_t>(bh) * nb + ib;
      warp_select_row(sm.keys + warp * nb, nb, p.pb, p.k_pre, p.k_gen, sm.hist + warp * 256, p.col_idx + r * k_total, lane);
      if (lane == 0) {
        p.row_ptr[r] = static_cast<int32_t>(r * k_total);
        if (r == static_cast<int64_t>(p.bh) * nb - 1) p.row_ptr[r + 1] = static_cast<int32_t>((r + 1) * k_total);
      }
    }
  }
}

}  // namespace

int pool_select_max_blocks() { return kMaxBlocks; }

cudaError_t launch_pool_select(const PoolParams& p, cudaStream_t stream) {
  const int nb = p.seq_len / p.block_size;
  if (nb > kMaxBlocks) return cudaErrorInvalidValue;
  const int smem = static_cast<int>(pool_smem_bytes(nb, kRows / p.block_size));
  static SmemLimit limit;
  cudaError_t e = ensure_dynamic_smem(pool_select_kernel, smem, limit);
  if (e != cudaSuccess) return e;
  const int num_q_tiles = (p.seq_len + kRows - 1) / kRows;
  const long long ctas = static_cast<long long>(p.bh) * num_q_tiles;
  if (ctas <= 0) return cudaSuccess;
  pool_select_kernel<<<static_cast<unsigned>(ctas), kRows, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace sparsed
