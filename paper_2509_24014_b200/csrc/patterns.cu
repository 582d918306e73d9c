// Fixed block patterns in the same CSR form the selected patterns use: a symmetric sliding
// window around the diagonal plus optional leading "sink" blocks. These are the sliding-window
// and StreamingLLM-style comparison patterns of the paper's experiments, expressed as block
// lists so that they run through the same block-sparse attention kernel.
#include "internal.h"

namespace sparsed {
namespace {

// kept blocks of query block i: [0, sink) united with [i - half, i + half] clipped to [0, nb)
__device__ __forceinline__ int window_row_count(int i, int nb, int sink, int half) {
  const int a = max(0, i - half), b = min(nb - 1, i + half);
  const int overlap = max(0, min(b, sink - 1) - a + 1);
  return (b - a + 1) + sink - overlap;
}

__global__ void __launch_bounds__(256) window_pattern_kernel(int32_t* row_ptr, int32_t* col_idx, int nb, int sink,
                                                            int half, int per_head_nnz, int bh_total) {
  __shared__ int partial[256];
  const int bh = blockIdx.x;
  const int tid = threadIdx.x;
  const int per = (nb + 255) / 256;
  const int r0 = min(nb, tid * per), r1 = min(nb, r0 + per);
  int local = 0;
  for (int i = r0; i < r1; ++i) local += window_row_count(i, nb, sink, half);
  partial[tid] = local;
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int t = 0; t < 256; ++t) {
      const int v = partial[t];
      partial[t] = run;
      run += v;
    }
  }
  __syncthreads();
  int offset = bh * per_head_nnz + partial[tid];
  for (int i = r0; i < r1; ++i) {
    row_ptr[bh * nb + i] = offset;
    const int a = max(0, i - half), b = min(nb - 1, i + half);
    for (int j = 0; j < min(sink, a); ++j) col_idx[offset++] = j;   // sink blocks below the window
    for (int j = a; j <= b; ++j) col_idx[offset++] = j;             // the window
    for (int j = max(b + 1, 0); j < sink; ++j) col_idx[offset++] = j;  // sink blocks above the window
  }
  if (bh == bh_total - 1 && tid == 0) row_ptr[bh_total * nb] = bh_total * per_head_nnz;
}

}  // namespace

int64_t window_pattern_nnz_per_head(int nb, int sink, int half) {
  int64_t total = 0;
  for (int i = 0; i < nb; ++i) {
    const int a = i - half > 0 ? i - half : 0, b = i + half < nb - 1 ? i + half : nb - 1;
    const int top = (b < sink - 1 ? b : sink - 1);
    const int overlap = top - a + 1 > 0 ? top - a + 1 : 0;
    total += (b - a + 1) + sink - overlap;
  }
  return total;
}

cudaError_t launch_window_pattern(int32_t* row_ptr, int32_t* col_idx, int bh, int nb, int sink, int half,
                                  int per_head_nnz, cudaStream_t stream) {
  if (bh <= 0) return cudaSuccess;
  window_pattern_kernel<<<bh, 256, 0, stream>>>(row_ptr, col_idx, nb, sink, half, per_head_nnz, bh);
  return cudaGetLastError();
}

}  // namespace sparsed
