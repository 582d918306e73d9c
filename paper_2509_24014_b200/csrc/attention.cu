// Dense bidirectional attention (Eq. 1 times V) and block-sparse attention (Eq. 3 / Eq. 4
// times V) for head_dim 128, bf16 in / bf16 out, fp32 softmax, on sm_100a.
//
// One CTA owns one query tile of one (batch, head) and streams key/value tiles through a
// warp-specialised pipeline:
//   warp 4  : TMA producer  - Q once, then a K tile and a V tile per step (128B-swizzled smem)
//   warp 5  : UMMA issuer   - S = Q K^T into tensor memory, then O += P V with P read from
//                             tensor memory (P overwrites the first half of S's columns)
//   warps 0-3: one thread per query row - online softmax in fp32 on the scaled base-2 logits,
//             writes P as bf16 into tensor memory, rescales O only when the running row
//             maximum grew by more than 2^8, and finally normalises and stores O (and LSE).
// The dense kernel walks all key tiles; the sparse kernel walks the CSR list of its query
// block. Two CTAs fit on one SM (96 KB of shared memory, 256 tensor-memory columns each), so
// one CTA's softmax overlaps the other's tensor-core work.
#include "internal.h"

namespace sparsed {
namespace {

constexpr int kHeadDim = 128;
constexpr int kTileM = 128;        // UMMA M; rows of tensor memory
constexpr int kSoftmaxThreads = 128;
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;
constexpr int kColS = 0;           // S (fp32) and P (bf16 pairs) live here
constexpr int kColO = 128;         // O accumulator (fp32)
constexpr float kRescaleThreshold = 8.0f;  // in log2 units

template <int kBlockN>
struct AttnSmem {
  alignas(1024) __nv_bfloat16 q[2][kTileM * 64];
  alignas(1024) __nv_bfloat16 k[2][kBlockN * 64];
  alignas(1024) __nv_bfloat16 v[2][kBlockN * 64];
  uint64_t q_full, k_full, k_empty, v_full, v_empty, s_full, p_full, o_full;
  uint32_t tmem_base;
  int abort_flag;
};

// kBlockN : keys per tile (64 or 128).  kRowsQ : valid query rows per tile (64 or 128).
template <int kBlockN, int kRowsQ, bool kSparse>
__global__ void __launch_bounds__(kThreads, 2)
attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
            const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  using Smem = AttnSmem<kBlockN>;
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  // ---- work item -----------------------------------------------------------------------
  const int q_tile = blockIdx.x % p.num_q_tiles;
  const int bh = blockIdx.x / p.num_q_tiles;
  const int head = bh % p.heads_q;
  const int batch = bh / p.heads_q;
  const int kv_head = head / p.group;
  const int q_row0 = q_tile * kRowsQ;

  int tile_begin = 0, num_tiles;
  if constexpr (kSparse) {
    const int r = bh * p.num_q_tiles + q_tile;
    tile_begin = __ldg(p.row_ptr + r);
    num_tiles = __ldg(p.row_ptr + r + 1) - tile_begin;
  } else {
    num_tiles = (p.seq_len + kBlockN - 1) / kBlockN;
  }

  // ---- set-up --------------------------------------------------------------------------
  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    mbar_init(&sm.k_full, 1);
    mbar_init(&sm.k_empty, 1);
    mbar_init(&sm.v_full, 1);
    mbar_init(&sm.v_empty, 1);
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.p_full, kSoftmaxThreads);
    mbar_init(&sm.o_full, 1);
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  if constexpr (kRowsQ < kTileM) {
    // rows the TMA box does not cover are multiplied too: keep them finite (zero)
    uint4* z0 = reinterpret_cast<uint4*>(&sm.q[0][kRowsQ * 64]);
    uint4* z1 = reinterpret_cast<uint4*>(&sm.q[1][kRowsQ * 64]);
    constexpr int n16 = (kTileM - kRowsQ) * 64 * 2 / 16;
    for (int i = tid; i < n16; i += kThreads) {
      z0[i] = make_uint4(0, 0, 0, 0);
      z1[i] = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
  }
  if (warp == 5) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tS = tmem + kColS;
  const uint32_t tO = tmem + kColO;

  if (warp == 4) {
    // =============================== TMA producer =======================================
    if (lane == 0 && num_tiles > 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      mbar_expect_tx(&sm.q_full, kRowsQ * kHeadDim * 2);
      tma_load_4d(sm.q[0], &tm_q, &sm.q_full, 0, q_row0, head, batch);
      tma_load_4d(sm.q[1], &tm_q, &sm.q_full, 64, q_row0, head, batch);
      for (int it = 0; it < num_tiles; ++it) {
        int kv_tile;
        if constexpr (kSparse) kv_tile = __ldg(p.col_idx + tile_begin + it);
        else kv_tile = it;
        const int kv_row0 = kv_tile * kBlockN;
        if (it > 0 && !mbar_wait(&sm.k_empty, (it - 1) & 1, &sm.abort_flag, p.status, 10)) break;
        mbar_expect_tx(&sm.k_full, kBlockN * kHeadDim * 2);
        tma_load_4d(sm.k[0], &tm_k, &sm.k_full, 0, kv_row0, kv_head, batch);
        tma_load_4d(sm.k[1], &tm_k, &sm.k_full, 64, kv_row0, kv_head, batch);
        if (it > 0 && !mbar_wait(&sm.v_empty, (it - 1) & 1, &sm.abort_flag, p.status, 11)) break;
        mbar_expect_tx(&sm.v_full, kBlockN * kHeadDim * 2);
        tma_load_4d(sm.v[0], &tm_v, &sm.v_full, 0, kv_row0, kv_head, batch);
        tma_load_4d(sm.v[1], &tm_v, &sm.v_full, 64, kv_row0, kv_head, batch);
      }
    }
  } else if (warp == 5) {
    // =============================== UMMA issuer ========================================
    if (lane == 0 && num_tiles > 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(kTileM, kBlockN, false, false);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(kTileM, kHeadDim, false, true);
      const uint32_t q_addr[2] = {smem_u32(sm.q[0]), smem_u32(sm.q[1])};
      const uint32_t k_addr[2] = {smem_u32(sm.k[0]), smem_u32(sm.k[1])};
      const uint32_t v_addr = smem_u32(sm.v[0]);
      bool ok = mbar_wait(&sm.q_full, 0, &sm.abort_flag, p.status, 20);
      for (int it = 0; ok && it < num_tiles; ++it) {
        const uint32_t ph = it & 1;
        if (!mbar_wait(&sm.k_full, ph, &sm.abort_flag, p.status, 21)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kHeadDim / 16; ++kk) {
          const uint32_t off = (kk & 3) * 32;
          umma_ss(tS, umma_smem_desc_sw128(q_addr[kk >> 2] + off, 16, 1024),
                  umma_smem_desc_sw128(k_addr[kk >> 2] + off, 16, 1024), idesc_qk, kk > 0);
        }
        umma_commit(&sm.k_empty);
        umma_commit(&sm.s_full);
        if (!mbar_wait(&sm.p_full, ph, &sm.abort_flag, p.status, 22)) break;
        if (!mbar_wait(&sm.v_full, ph, &sm.abort_flag, p.status, 23)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kBlockN / 16; ++kk) {
          // V tile is [key][d]: MN-major B operand; 64-wide d halves are kBlockN*128 bytes apart
          umma_ts(tO, tS + kk * 8, umma_smem_desc_sw128(v_addr + kk * 2048, kBlockN * 128, 1024), idesc_pv,
                  (it > 0) || (kk > 0));
        }
        umma_commit(&sm.v_empty);
        if (it == num_tiles - 1) umma_commit(&sm.o_full);
      }
    }
  } else {
    // =============================== softmax / epilogue =================================
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const float scale_log2 = p.scale_log2;
    float m_used = -INFINITY;
    float l = 0.f;
    bool ok = true;
    for (int it = 0; it < num_tiles; ++it) {
      if (!mbar_wait(&sm.s_full, it & 1, &sm.abort_flag, p.status, 30)) {
        ok = false;
        break;
      }
      tc_fence_after();
      int valid_cols = kBlockN;
      if constexpr (!kSparse) {
        if (it == num_tiles - 1) valid_cols = p.seq_len - it * kBlockN;
      }
      // pass 1: row maximum of the raw logits of this tile
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < kBlockN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tS + lane_base + c * 32, r);
        tmem_wait_ld();
        if (valid_cols >= (c + 1) * 32) {
#pragma unroll
          for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(r[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j < valid_cols) mx = fmaxf(mx, __uint_as_float(r[j]));
        }
      }
      const float m_tile = mx * scale_log2;
      bool need = false;
      float alpha = 1.f;
      if (it == 0) {
        m_used = m_tile;
      } else {
        need = (m_tile - m_used) > kRescaleThreshold;
      }
      const bool any_need = __any_sync(0xffffffffu, need);
      if (need) {
        alpha = fast_exp2(m_used - m_tile);
        m_used = m_tile;
        l *= alpha;
      }
      // pass 2: p = 2^(s*scale - m), row sum, bf16 P into tensor memory (over S's first columns)
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < kBlockN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tS + lane_base + c * 32, r);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float p0 = fast_exp2(fmaf(__uint_as_float(r[2 * j]), scale_log2, -m_used));
          float p1 = fast_exp2(fmaf(__uint_as_float(r[2 * j + 1]), scale_log2, -m_used));
          if constexpr (!kSparse) {
            if (c * 32 + 2 * j >= valid_cols) p0 = 0.f;
            if (c * 32 + 2 * j + 1 >= valid_cols) p1 = 0.f;
          }
          sum += p0;
          sum += p1;
          pk[j] = pack_bf16x2(p0, p1);
        }
        tmem_st16(tS + lane_base + c * 16, pk);
      }
      l += sum;
      if (any_need) {
        // the previous P V finished before this tile's S was signalled, so O is quiescent
#pragma unroll
        for (int c = 0; c < kHeadDim / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tO + lane_base + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
          tmem_st32(tO + lane_base + c * 32, r);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sm.p_full);
    }

    // ---- epilogue: O / l -> bf16 -> global; LSE ----------------------------------------
    if (ok && num_tiles > 0) ok = mbar_wait(&sm.o_full, 0, &sm.abort_flag, p.status, 31);
    tc_fence_after();
    const int row_in_tile = tid;
    const int row = q_row0 + row_in_tile;
    const bool row_valid = (row_in_tile < kRowsQ) && (row < p.seq_len);
    const float inv_l = (num_tiles > 0) ? (1.f / l) : 0.f;
    __nv_bfloat16* o_row = reinterpret_cast<__nv_bfloat16*>(p.o) + batch * p.o_stride_b + head * p.o_stride_h +
                           static_cast<int64_t>(row) * p.o_stride_t;
#pragma unroll
    for (int c = 0; c < kHeadDim / 32; ++c) {
      uint32_t r[32];
      if (num_tiles > 0) {
        tmem_ld32(tO + lane_base + c * 32, r);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = 0u;
      }
      if (row_valid) {
        uint4* dst = reinterpret_cast<uint4*>(o_row + c * 32);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint4 out;
          out.x = pack_bf16x2(__uint_as_float(r[8 * g + 0]) * inv_l, __uint_as_float(r[8 * g + 1]) * inv_l);
          out.y = pack_bf16x2(__uint_as_float(r[8 * g + 2]) * inv_l, __uint_as_float(r[8 * g + 3]) * inv_l);
          out.z = pack_bf16x2(__uint_as_float(r[8 * g + 4]) * inv_l, __uint_as_float(r[8 * g + 5]) * inv_l);
          out.w = pack_bf16x2(__uint_as_float(r[8 * g + 6]) * inv_l, __uint_as_float(r[8 * g + 7]) * inv_l);
          dst[g] = out;
        }
      }
    }
    if (p.lse != nullptr && row_valid) {
      const float lse = (num_tiles > 0) ? (m_used + log2f(l)) * 0.69314718055994531f : -INFINITY;
      p.lse[static_cast<int64_t>(bh) * p.seq_len + row] = lse;
    }
  }

  // ---- teardown ------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int kBlockN, int kRowsQ, bool kSparse>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                   int batch, cudaStream_t stream) {
  auto kernel = attn_kernel<kBlockN, kRowsQ, kSparse>;
  const int smem = static_cast<int>(sizeof(AttnSmem<kBlockN>)) + 1024;
  static bool configured[64] = {};  // per template instantiation and device
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const long long ctas = static_cast<long long>(batch) * p.heads_q * p.num_q_tiles;
  if (ctas <= 0) return cudaSuccess;
  kernel<<<static_cast<unsigned>(ctas), kThreads, smem, stream>>>(tq, tk, tv, p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_dense(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                              const AttnParams& p, int batch, cudaStream_t stream) {
  return launch<128, 128, false>(tq, tk, tv, p, batch, stream);
}

cudaError_t launch_attn_sparse(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const AttnParams& p, int batch, int block_size, cudaStream_t stream) {
  if (block_size == 128) return launch<128, 128, true>(tq, tk, tv, p, batch, stream);
  return launch<64, 64, true>(tq, tk, tv, p, batch, stream);
}

}  // namespace sparsed
