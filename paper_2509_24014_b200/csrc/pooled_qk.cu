// Block-mean estimate of the pooled scores A' and selection from it.
//
// This is NOT the paper's scorer. The paper pools the exact post-softmax probabilities; the
// family of methods it sets itself against estimates block importance from pooled queries and
// keys. This file builds that estimate so that its recall of the exact pattern (and its cost)
// can be measured on the same inputs:
//
//   mean_q[i] = mean of the rows of query block i,  mean_k[j] = mean of the rows of key block j
//   est[i][j] = softmax_j(scale * mean_q[i] . mean_k[j]) / block_size
//
// followed by the same isolated top-rho% selection (Eq. 5 / Eq. 6) and CSR compaction.
//
// Two kernels, both bandwidth / ALU work with no dense contraction worth a tensor-core tile
// (nb x nb x 128 multiply-adds per head, 0.06 % of the exact scorer's):
//   block_mean_kernel        one CTA per (block, head, batch): 16-byte loads, fp32 sums
//   pooled_qk_select_kernel  one CTA per 32 query blocks of a head: fp32 logits against all key
//                            blocks through shared-memory tiles, softmax, radix-select top-k
#include "internal.h"
#include "topk_device.cuh"

namespace sparsed {

namespace {

constexpr int kD = 128;

// ---------------------------------------------------------------------------------------------
// mean over the block_size rows of one block; x is bf16 with element strides (batch, head, token)
__global__ void __launch_bounds__(128)
block_mean_kernel(const __nv_bfloat16* __restrict__ x, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                  float* __restrict__ out, int heads, int nb, int block_size) {
  __shared__ float red[8][kD];
  const int blk = blockIdx.x, head = blockIdx.y, batch = blockIdx.z;
  const int tid = threadIdx.x;
  const int chunk = tid & 15;  // which 16 bytes (8 elements) of the 256-byte row
  const int r0 = tid >> 4;     // rows r0, r0 + 8, ...
  const __nv_bfloat16* base = x + batch * stride_b + head * stride_h +
                              static_cast<int64_t>(blk) * block_size * stride_t + chunk * 8;
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll 4
  for (int r = r0; r < block_size; r += 8) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(base + r * stride_t));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[2 * e] += __uint_as_float(w[e] << 16);
      acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[r0][chunk * 8 + e] = acc[e];
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int r = 0; r < 8; ++r) s += red[r][tid];
  out[((static_cast<int64_t>(batch) * heads + head) * nb + blk) * kD + tid] = s / static_cast<float>(block_size);
}

// ---------------------------------------------------------------------------------------------
constexpr int kRowsPerCta = 32;  // query blocks per CTA
constexpr int kColsPerTile = 64; // key blocks per shared-memory tile
constexpr int kPitch = kD + 4;   // floats per staged row: keeps 16-byte alignment, spreads banks

struct SelectSmemLayout {
  // floats: q tile, k tile, then the logits [kRowsPerCta][nb_pitch]; ints: 4 x 256 histogram bins
  static __host__ __device__ size_t bytes(int nb) {
    const size_t nb_pitch = static_cast<size_t>(nb + 3) / 4 * 4 + 4;
    return (static_cast<size_t>(kRowsPerCta + kColsPerTile) * kPitch + kRowsPerCta * nb_pitch) * 4 + 4 * 256 * 4;
  }
};

__global__ void __launch_bounds__(128)
pooled_qk_select_kernel(const float* __restrict__ mean_q, const float* __restrict__ mean_k, float* __restrict__ scores,
                        int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx, int heads_q, int group, int nb,
                        int pb, int k_pre, int k_gen, float scale_log2, float inv_block) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  float* qs = reinterpret_cast<float*>(smem_raw);            // [32][kPitch]
  float* ks = qs + kRowsPerCta * kPitch;                     // [64][kPitch]
  float* lg = ks + kColsPerTile * kPitch;                    // [32][nb_pitch]
  const int nb_pitch = (nb + 3) / 4 * 4 + 4;
  int* hist = reinterpret_cast<int*>(lg + kRowsPerCta * nb_pitch);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row_tiles = (nb + kRowsPerCta - 1) / kRowsPerCta;
  const int bh = blockIdx.x / row_tiles;
  const int i0 = (blockIdx.x % row_tiles) * kRowsPerCta;
  const int batch = bh / heads_q, head = bh % heads_q;
  const float* qsrc = mean_q + (static_cast<int64_t>(bh) * nb + i0) * kD;
  const float* ksrc = mean_k + (static_cast<int64_t>(batch) * (heads_q / group) + head / group) * nb * kD;

  // stage the query means (rows past nb read as zero)
  for (int idx = tid; idx < kRowsPerCta * (kD / 4); idx += 128) {
    const int r = idx / (kD / 4), c = idx % (kD / 4);
    float4 vq = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < nb) vq = __ldg(reinterpret_cast<const float4*>(qsrc + r * kD) + c);
    *reinterpret_cast<float4*>(qs + r * kPitch + c * 4) = vq;
  }

  // each thread: 4 query rows x 4 key columns of the tile
  const int ti = tid >> 4;  // rows 4 ti .. 4 ti + 3
  const int tj = tid & 15;  // columns tj, tj + 16, tj + 32, tj + 48
  const int n_tiles = (nb + kColsPerTile - 1) / kColsPerTile;
  float4 pre[16];
  auto fetch = [&](int jt) {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int idx = tid + u * 128;  // 64 rows x 32 float4
      const int r = idx >> 5, c = idx & 31;
      const int j = jt * kColsPerTile + r;
      pre[u] = j < nb ? __ldg(reinterpret_cast<const float4*>(ksrc + static_cast<int64_t>(j) * kD) + c)
                      : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  fetch(0);
  for (int jt = 0; jt < n_tiles; ++jt) {
    __syncthreads();  // the previous tile has been consumed (and, first time, qs is written)
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int idx = tid + u * 128;
      *reinterpret_cast<float4*>(ks + (idx >> 5) * kPitch + (idx & 31) * 4) = pre[u];
    }
    __syncthreads();
    if (jt + 1 < n_tiles) fetch(jt + 1);  // in flight while this tile is multiplied
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
    for (int d = 0; d < kD; d += 4) {
      float4 qa[4], kb[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) qa[a] = *reinterpret_cast<const float4*>(qs + (4 * ti + a) * kPitch + d);
#pragma unroll
      for (int b = 0; b < 4; ++b) kb[b] = *reinterpret_cast<const float4*>(ks + (tj + 16 * b) * kPitch + d);
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          acc[a][b] = fmaf(qa[a].x, kb[b].x, acc[a][b]);
          acc[a][b] = fmaf(qa[a].y, kb[b].y, acc[a][b]);
          acc[a][b] = fmaf(qa[a].z, kb[b].z, acc[a][b]);
          acc[a][b] = fmaf(qa[a].w, kb[b].w, acc[a][b]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int j = jt * kColsPerTile + tj + 16 * b;
        if (j < nb) lg[(4 * ti + a) * nb_pitch + j] = acc[a][b] * scale_log2;  // base-2 logits
      }
  }
  __syncthreads();

  // softmax over the nb key blocks, estimate = p / block_size, then the isolated top-k; one warp per row
  int* my_hist = hist + warp * 256;
  const int k_total = k_pre + k_gen;
  for (int r = warp; r < kRowsPerCta; r += 4) {
    const int i = i0 + r;
    if (i >= nb) break;
    float* row = lg + r * nb_pitch;
    float m = -INFINITY;
    for (int j = lane; j < nb; j += 32) m = fmaxf(m, row[j]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float sum = 0.f;
    for (int j = lane; j < nb; j += 32) {
      const float e = exp2f(row[j] - m);
      row[j] = e;
      sum += e;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const float norm = inv_block / sum;
    const int64_t grow = static_cast<int64_t>(bh) * nb + i;
    uint32_t* keys = reinterpret_cast<uint32_t*>(row);
    for (int j = lane; j < nb; j += 32) {
      const float est = row[j] * norm;
      if (scores != nullptr) scores[grow * nb + j] = est;
      keys[j] = ordered_key(est);
    }
    __syncwarp();
    warp_select_row(keys, nb, pb, k_pre, k_gen, my_hist, col_idx + grow * k_total, lane);
    if (lane == 0) {
      row_ptr[grow + 1] = static_cast<int32_t>((grow + 1) * k_total);
      if (grow == 0) row_ptr[0] = 0;
    }
    __syncwarp();
  }
}

}  // namespace

size_t pooled_qk_means_bytes(int batch, int heads_q, int heads_kv, int nb) {
  return static_cast<size_t>(batch) * (heads_q + heads_kv) * nb * kD * sizeof(float);
}

cudaError_t launch_pooled_qk_select(const PooledQkParams& p, cudaStream_t stream) {
  const int heads_kv = p.heads_q / p.group;
  float* mean_q = p.means;
  float* mean_k = p.means + static_cast<size_t>(p.batch) * p.heads_q * p.nb * kD;
  block_mean_kernel<<<dim3(p.nb, p.heads_q, p.batch), 128, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(p.q), p.q_stride_b, p.q_stride_h, p.q_stride_t, mean_q, p.heads_q, p.nb,
      p.block_size);
  block_mean_kernel<<<dim3(p.nb, heads_kv, p.batch), 128, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(p.k), p.k_stride_b, p.k_stride_h, p.k_stride_t, mean_k, heads_kv, p.nb,
      p.block_size);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = SelectSmemLayout::bytes(p.nb);
  if (smem > 48 * 1024) {
    static SmemLimit limit;
    e = ensure_dynamic_smem(pooled_qk_select_kernel, static_cast<int>(smem), limit);
    if (e != cudaSuccess) return e;
  }
  const int row_tiles = (p.nb + kRowsPerCta - 1) / kRowsPerCta;
  pooled_qk_select_kernel<<<p.batch * p.heads_q * row_tiles, 128, smem, stream>>>(
      mean_q, mean_k, p.scores, p.row_ptr, p.col_idx, p.heads_q, p.group, p.nb, p.pb, p.k_pre, p.k_gen, p.scale_log2,
      1.0f / static_cast<float>(p.block_size));
  return cudaGetLastError();
}

}  // namespace sparsed
