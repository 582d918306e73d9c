// Per-row isolated top-k over pooled block scores and compaction into CSR block lists
// (Eq. 5 / Eq. 6; the IndexSelection and mask-write lines of Algorithm 1).
//
// One warp owns one row (batch, head, query block) of A'. The row's nb fp32 scores are read
// once, coalesced, into registers as order-preserving 32-bit keys. For each key region
// (prefill blocks [0,pb), generation blocks [pb,nb)) the k-th largest key is found by a
// 32-step bitwise search with warp-wide counts; blocks above it are kept, blocks equal to
// it are kept lowest index first until k are kept (ties -> lower block index). Kept ids are
// written in ascending order through ballot prefix sums. Every row keeps the same number of
// blocks, so row_ptr is an arithmetic sequence written by the same kernel.
// HBM-bound by design: 4*nb bytes read and 4*(k_pre+k_gen) + 4 bytes written per row.
#include "internal.h"

namespace sparsed {
namespace {

// Order-preserving map float -> uint32 (larger float -> larger key). NaN ranks lowest,
// -0 equals +0.
__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;  // NaN
  if (u == 0x80000000u) u = 0u;                    // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int kSlots>
__global__ void __launch_bounds__(256) topk_csr_kernel(const TopkParams p) {
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp_global >= p.rows) return;
  const int row = warp_global;
  const float* src = p.scores + static_cast<int64_t>(row) * p.nb;
  const int k_total = p.k_pre + p.k_gen;

  uint32_t key[kSlots];
#pragma unroll
  for (int t = 0; t < kSlots; ++t) {
    const int idx = t * 32 + lane;
    key[t] = (idx < p.nb) ? ordered_key(__ldg(src + idx)) : 0u;
  }

  uint32_t keep_mask = 0;  // bit t: this lane's slot t is kept (kSlots <= 32)
#pragma unroll 1
  for (int region = 0; region < 2; ++region) {
    const int lo = region == 0 ? 0 : p.pb;
    const int hi = region == 0 ? p.pb : p.nb;
    const int kk = region == 0 ? p.k_pre : p.k_gen;
    if (hi <= lo || kk <= 0) continue;
    uint32_t in_region = 0;
#pragma unroll
    for (int t = 0; t < kSlots; ++t) {
      const int idx = t * 32 + lane;
      if (idx >= lo && idx < hi) in_region |= (1u << t);
    }
    // largest T with count(key >= T) >= kk  ==  the kk-th largest key of the region
    uint32_t thr = 0;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
      const uint32_t cand = thr | (1u << bit);
      int cnt = 0;
#pragma unroll
      for (int t = 0; t < kSlots; ++t) cnt += ((in_region >> t) & 1u) && (key[t] >= cand);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (cnt >= kk) thr = cand;
    }
    int n_gt = 0;
#pragma unroll
    for (int t = 0; t < kSlots; ++t) n_gt += ((in_region >> t) & 1u) && (key[t] > thr);
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    const int need_eq = kk - n_gt;  // >= 1
    int eq_before = 0;              // equal keys at lower block indices (slot-major = index order)
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int t = 0; t < kSlots; ++t) {
      const bool in_r = (in_region >> t) & 1u;
      const bool eq = in_r && (key[t] == thr);
      const uint32_t b = __ballot_sync(0xffffffffu, eq);
      const int rank = eq_before + __popc(b & lt_mask);
      if (in_r && (key[t] > thr || (eq && rank < need_eq))) keep_mask |= (1u << t);
      eq_before += __popc(b);
    }
  }

  // ordered compaction: block ids ascending
  int32_t* dst = p.col_idx + static_cast<int64_t>(row) * k_total;
  int run = 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int t = 0; t < kSlots; ++t) {
    const bool kp = (keep_mask >> t) & 1u;
    const uint32_t b = __ballot_sync(0xffffffffu, kp);
    if (kp) dst[run + __popc(b & lt_mask)] = t * 32 + lane;
    run += __popc(b);
  }
  if (lane == 0) {
    p.row_ptr[row] = row * k_total;
    if (row == p.rows - 1) p.row_ptr[p.rows] = p.rows * k_total;
  }
}

__global__ void pattern_validate_kernel(const int32_t* row_ptr, const int32_t* col_idx, int rows, int nb,
                                        int64_t capacity, int* bad_flag) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const int64_t a = row_ptr[r], b = row_ptr[r + 1];
  bool bad = (a < 0) || (b <= a) || (b > capacity) || (r == 0 && a != 0);
  if (!bad) {
    int prev = -1;
    for (int64_t i = a; i < b; ++i) {
      const int c = col_idx[i];
      if (c <= prev || c >= nb) {
        bad = true;
        break;
      }
      prev = c;
    }
  }
  if (bad) atomicExch(bad_flag, r + 1);
}

}  // namespace

cudaError_t launch_topk_csr(const TopkParams& p, cudaStream_t stream) {
  if (p.rows <= 0) return cudaSuccess;
  const int threads = 256;
  const int warps_per_cta = threads / 32;
  const unsigned ctas = static_cast<unsigned>((p.rows + warps_per_cta - 1) / warps_per_cta);
  const int slots = (p.nb + 31) / 32;
  if (slots <= 1) topk_csr_kernel<1><<<ctas, threads, 0, stream>>>(p);
  else if (slots <= 2) topk_csr_kernel<2><<<ctas, threads, 0, stream>>>(p);
  else if (slots <= 4) topk_csr_kernel<4><<<ctas, threads, 0, stream>>>(p);
  else if (slots <= 8) topk_csr_kernel<8><<<ctas, threads, 0, stream>>>(p);
  else if (slots <= 16) topk_csr_kernel<16><<<ctas, threads, 0, stream>>>(p);
  else if (slots <= 32) topk_csr_kernel<32><<<ctas, threads, 0, stream>>>(p);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

cudaError_t launch_pattern_validate(const int32_t* row_ptr, const int32_t* col_idx, int rows, int nb,
                                    int64_t capacity, int* bad_flag, cudaStream_t stream) {
  if (rows <= 0) return cudaSuccess;
  pattern_validate_kernel<<<(rows + 255) / 256, 256, 0, stream>>>(row_ptr, col_idx, rows, nb, capacity, bad_flag);
  return cudaGetLastError();
}

}  // namespace sparsed
