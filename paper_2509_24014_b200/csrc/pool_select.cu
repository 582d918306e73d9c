// Pattern selection from the row statistics of the switch step's full-attention pass
// ("Isolated Selection": A' = avgpool(A, block_size), then Eq. 5 / Eq. 6), without a second
// Q K^T pass.
//
// The dense attention kernel can record, for every query row i and every 64-key tile t,
// v[t][i] = log2 sum_{j in t} 2^(s_ij), the tile's share of the row's softmax denominator.
// With the row's final log-sum-exp, 2^(v[t][i] - LSE_i) is exactly the probability mass row i
// puts on tile t, so A'[ib][jb] is the sum of that mass over the rows of block ib and the tiles
// of block jb, divided by block_size^2.
//
// One CTA owns one 128-row query tile of one (batch, head). Statistics are read with 16-byte
// loads (four consecutive rows of one tile; the layout [bh][128-row query tile][key tile][row]
// makes a CTA's reads one contiguous run), eight in flight per thread and six CTAs per SM (the
// best point of a sweep: 5.9 TB/s at 64k), exponentiated, parked in shared memory in chunks of 32
// tiles, and summed per tile and row half in a fixed, bank-conflict-free order (bitwise
// reproducible); the next chunk's loads are issued before the current chunk is summed.
// The CTA then holds its block-row(s) of A' in shared memory, optionally writes them out, and
// warp 0 ranks them (warp_select_row) and writes the CSR lists. HBM-bound:
// 4 * 128 * ceil(L/128) * ceil(L/64) bytes read per (batch, head).
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
constexpr int kMaxTiles = 2048;     // seq_len <= 131072

// Shared memory (dynamic, sized for the actual sequence): the transposition chunk, the per-tile
// mass of rows 0-63 / 64-127, the ordered keys of this CTA's block-row(s), the top-k histogram.
struct PoolSmem {
  float* chunk;                     // [tile in chunk][kPitch]
  float* tile_sum[2];               // [row half][tile]
  uint32_t* keys[2];
  int* hist;
};

__host__ __device__ inline size_t pool_smem_bytes(int n_tiles, int nb) {
  return sizeof(float) * kChunk * kPitch + sizeof(float) * 2 * n_tiles + sizeof(uint32_t) * 2 * nb +
         sizeof(int) * 256;
}

__global__ void __launch_bounds__(kRows, SPARSED_POOL_CTAS_PER_SM) pool_select_kernel(const PoolParams p) {
  extern __shared__ __align__(16) uint8_t pool_smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = p.seq_len;
  const int n_tiles = (L + 63) / 64;
  PoolSmem sm;
  {
    float* f = reinterpret_cast<float*>(pool_smem_raw);
    sm.chunk = f;
    f += kChunk * kPitch;
    sm.tile_sum[0] = f;
    sm.tile_sum[1] = f + n_tiles;
    f += 2 * n_tiles;
    const int nb_ = L / p.block_size;
    sm.keys[0] = reinterpret_cast<uint32_t*>(f);
    sm.keys[1] = sm.keys[0] + nb_;
    sm.hist = reinterpret_cast<int*>(sm.keys[1] + nb_);
  }
  const int num_q_tiles = (L + kRows - 1) / kRows;
  const int q_tile = blockIdx.x % num_q_tiles;
  const int bh = blockIdx.x / num_q_tiles;
  // Loading: lane l owns rows 4l..4l+3 of the query tile (one 16-byte load covers them), warp w
  // takes tiles w, w+4, ... of the chunk. seq_len is a multiple of 32 here, so a group of four
  // rows is valid or invalid as a whole and 16-byte aligned.
  const int row4 = q_tile * kRows + lane * 4;
  const bool rows_valid = row4 < L;
  float4 lse2 = make_float4(INFINITY, INFINITY, INFINITY, INFINITY);
  if (rows_valid) {
    const float4 t = *reinterpret_cast<const float4*>(p.lse + static_cast<int64_t>(bh) * L + row4);
    const float c = 1.44269504088896341f;
    lse2 = make_float4(t.x * c, t.y * c, t.z * c, t.w * c);
  }
  // statistics layout [bh][query tile][key tile][128 rows]: this CTA's share is one contiguous run
  const float* src = p.tile_lse + (static_cast<int64_t>(bh) * num_q_tiles + q_tile) * n_tiles * kRows + lane * 4;

  // One batch = this thread's kInFlight loads of a chunk (warp w takes tiles w, w+4, ... of it). The
  // next chunk's batch is issued before the current chunk is summed, so loads stay in flight
  // through the shared-memory phase.
  static_assert(kChunk == 4 * kInFlight, "one batch of loads per thread covers one chunk");
  float4 v[kInFlight];
  auto issue = [&](int c0) {
    const int n_here = min(kChunk, n_tiles - c0);
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int t = warp + 4 * u;
      v[u] = (rows_valid && t < n_here)
                 ? __ldcs(reinterpret_cast<const float4*>(src + static_cast<int64_t>(c0 + t) * kRows))
                 : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
  };
  issue(0);
  for (int c0 = 0; c0 < n_tiles; c0 += kChunk) {
    const int n_here = min(kChunk, n_tiles - c0);
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
    if (c0 + kChunk < n_tiles) issue(c0 + kChunk);
    {
      // Summing: thread j < 64 adds rows 0-63 of tile j, thread j + 64 rows 64-127. Each thread
      // starts at its own rotation of the 64 rows so that a warp's reads hit 32 different banks;
      // the order is fixed per tile, so the result is reproducible.
      const int half = tid >> 6;
      for (int j = tid & 63; j < n_here; j += 64) {
        const float* rowp = sm.chunk + j * kPitch + half * 64;
        float acc = 0.f;
#pragma unroll 8
        for (int r = 0; r < 64; ++r) acc += rowp[(r + 29 * j) & 63];
        sm.tile_sum[half][c0 + j] = acc;
      }
    }
    __syncthreads();
  }

  const int bs = p.block_size;
  const int nb = L / bs;
  const float inv_area = 1.f / (static_cast<float>(bs) * static_cast<float>(bs));
  const int rows_here = bs == 64 ? 2 : 1;
  for (int jb = tid; jb < nb; jb += kRows) {
    if (bs == 128) {
      const float total = (sm.tile_sum[0][2 * jb] + sm.tile_sum[1][2 * jb]) +
                          (sm.tile_sum[0][2 * jb + 1] + sm.tile_sum[1][2 * jb + 1]);
      const float score = total * inv_area;
      sm.keys[0][jb] = ordered_key(score);
      if (p.scores != nullptr) p.scores[(static_cast<int64_t>(bh) * nb + q_tile) * nb + jb] = score;
    } else {
#pragma unroll
      for (int rh = 0; rh < 2; ++rh) {
        const int ib = q_tile * 2 + rh;
        if (ib < nb) {
          const float score = sm.tile_sum[rh][jb] * inv_area;
          sm.keys[rh][jb] = ordered_key(score);
          if (p.scores != nullptr) p.scores[(static_cast<int64_t>(bh) * nb + ib) * nb + jb] = score;
        }
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int k_total = p.k_pre + p.k_gen;
    for (int rh = 0; rh < rows_here; ++rh) {
      const int ib = bs == 64 ? q_tile * 2 + rh : q_tile;
      if (ib >= nb) break;
      const int64_t r = static_cast<int64_t>(bh) * nb + ib;
      warp_select_row(sm.keys[rh], nb, p.pb, p.k_pre, p.k_gen, sm.hist, p.col_idx + r * k_total, lane);
      if (lane == 0) {
        p.row_ptr[r] = static_cast<int32_t>(r * k_total);
        if (r == static_cast<int64_t>(p.bh) * nb - 1) p.row_ptr[r + 1] = static_cast<int32_t>((r + 1) * k_total);
      }
      __syncwarp();
    }
  }
}

}  // namespace

cudaError_t launch_pool_select(const PoolParams& p, cudaStream_t stream) {
  const int n_tiles = (p.seq_len + 63) / 64;
  if (n_tiles > kMaxTiles) return cudaErrorInvalidValue;
  const int smem = static_cast<int>(pool_smem_bytes(n_tiles, p.seq_len / p.block_size));
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
