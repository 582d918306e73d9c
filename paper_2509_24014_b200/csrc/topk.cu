// Per-row isolated top-k over pooled block scores and compaction into CSR block lists
// (Eq. 5 / Eq. 6; the IndexSelection and mask-write lines of Algorithm 1), as a kernel of
// its own for scores that already sit in memory.
//
// One warp owns one row (batch, head, query block) of A'. The row's nb fp32 scores are read
// once with coalesced 16-byte loads and parked in shared memory as order-preserving keys;
// the selection itself is warp_select_row (radix selection + ordered ballot compaction).
// Every row keeps the same number of blocks, so row_ptr is an arithmetic sequence written by
// the same kernel. HBM-bound by design: 4*nb bytes read and 4*(k_pre+k_gen) + 4 bytes
// written per row.
#include "internal.h"
#include "topk_device.cuh"

namespace sparsed {
namespace {

__global__ void __launch_bounds__(256) topk_csr_kernel(const TopkParams p, int warps_per_cta) {
  extern __shared__ __align__(16) uint8_t topk_smem[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * warps_per_cta + warp;
  if (warp >= warps_per_cta || row >= p.rows) return;
  const int nb_pad = (p.nb + 3) & ~3;
  uint32_t* keys = reinterpret_cast<uint32_t*>(topk_smem) + static_cast<size_t>(warp) * (nb_pad + 256);
  int* hist = reinterpret_cast<int*>(keys + nb_pad);
  const float* src = p.scores + static_cast<int64_t>(row) * p.nb;
  if ((p.nb & 3) == 0) {
    const float4* src4 = reinterpret_cast<const float4*>(src);
    for (int i = lane; i < p.nb / 4; i += 32) {
      const float4 v = __ldg(src4 + i);
      reinterpret_cast<uint4*>(keys)[i] = make_uint4(ordered_key(v.x), ordered_key(v.y), ordered_key(v.z), ordered_key(v.w));
    }
  } else {
    for (int i = lane; i < p.nb; i += 32) keys[i] = ordered_key(__ldg(src + i));
  }
  __syncwarp();
  const int k_total = p.k_pre + p.k_gen;
  warp_select_row(keys, p.nb, p.pb, p.k_pre, p.k_gen, hist, p.col_idx + static_cast<int64_t>(row) * k_total, lane);
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

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete, with
// a short poll limit, so the wait gives up, records {1, where} in the status word and the kernel
// returns normally.
__global__ void wait_timeout_selftest_kernel(DeviceStatus* status, int where, uint32_t limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  mbar_wait(&bar, 0, &abort_flag, status, where, limit);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(DeviceStatus* status, int where, cudaStream_t stream) {
  wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status, where, 1u << 12);
  return cudaGetLastError();
}

cudaError_t launch_topk_csr(const TopkParams& p, cudaStream_t stream) {
  if (p.rows <= 0) return cudaSuccess;
  if (p.nb > 16384) return cudaErrorInvalidValue;
  const int warps = p.nb <= 1024 ? 8 : (p.nb <= 4096 ? 4 : 2);
  const int nb_pad = (p.nb + 3) & ~3;
  const size_t smem = static_cast<size_t>(warps) * (nb_pad + 256) * 4;
  if (smem > 48 * 1024) {
    static SmemLimit limit;
    cudaError_t e = ensure_dynamic_smem(topk_csr_kernel, static_cast<int>(smem), limit);
    if (e != cudaSuccess) return e;
  }
  const unsigned ctas = static_cast<unsigned>((p.rows + warps - 1) / warps);
  topk_csr_kernel<<<ctas, warps * 32, smem, stream>>>(p, warps);
  return cudaGetLastError();
}

cudaError_t launch_pattern_validate(const int32_t* row_ptr, const int32_t* col_idx, int rows, int nb,
                                    int64_t capacity, int* bad_flag, cudaStream_t stream) {
  if (rows <= 0) return cudaSuccess;
  pattern_validate_kernel<<<(rows + 255) / 256, 256, 0, stream>>>(row_ptr, col_idx, rows, nb, capacity, bad_flag);
  return cudaGetLastError();
}

}  // namespace sparsed
