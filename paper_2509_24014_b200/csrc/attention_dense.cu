// Dense bidirectional attention (Eq. 1 times V; the full-attention branch of Algorithm 1) for
// head_dim 128, bf16 in / bf16 out, fp32 softmax, on sm_100a.
//
// One CTA per SM owns TWO consecutive 128-row query tiles of one (batch, head) and runs one
// pipeline of the block-sparse kernel's kind per tile ("stream"), side by side:
//   warp 8      : TMA producer - both Q tiles once, then every 64-key K tile and V tile ONCE for
//                 both streams into a nine-slot ring of 128B-swizzled shared memory (load 2t is
//                 K_t, load 2t+1 is V_t). Dense attention reads the same keys for every query tile,
//                 so sharing the ring halves the L2-to-SM traffic and the TMA work.
//   warps 9, 10 : UMMA issuer of stream 0 / 1 - S_t = Q K_t^T into one of the stream's two
//                 tensor-memory buffers, then O += P_t V_t with P read from tensor memory; S_{t+1}
//                 is issued before P_t V_t. A ring slot is released when both streams' MMAs that
//                 read it have completed (its barrier counts two arrivals).
//   warps 0-3, 4-7 : softmax warpgroup of stream 0 / 1, one thread per query row: the same
//                 single-pass online softmax with a stale running maximum as in the sparse kernel.
// The streams share nothing else (own S buffers, O accumulator, maxima), so they drift apart and
// one stream's softmax overlaps the other's MMAs. Tensor memory: 2 x (2 x 64 S + 128 O) = 512
// columns; shared memory 208 KB. Optional outputs: LSE, and the per-(row, 64-key tile) statistic
// m + log2(sum p) from which the switch step's pooled scores are formed (laid out
// [batch*head][128-row query tile][key tile][row], so that both this kernel's writes and the
// pooling kernel's reads are contiguous per query tile).
#include "internal.h"

namespace sparsed {
namespace {


constexpr int kHeadDim = 128;
constexpr int kTileM = 128;
constexpr int kTileN = 64;
constexpr int kSlots = 9;             // 16 KB each, shared by K and V: load 2t is K_t, load 2t+1 is V_t
constexpr int kThreads = 352;         // warps 0-3 softmax A, 4-7 softmax B, 8 TMA, 9 UMMA A, 10 UMMA B
constexpr int kTmemCols = 512;

struct PairSmem {
  alignas(1024) __nv_bfloat16 q[2][2][kTileM * 64];
  alignas(1024) __nv_bfloat16 kv[kSlots][2][kTileN * 64];
  uint64_t q_full[2], kv_full[kSlots], kv_empty[kSlots];
  uint64_t s_full[2][2], p_full[2][2], pv_done[2], o_full[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
attn_dense_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  PairSmem& sm = *reinterpret_cast<PairSmem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0u) {
    if (threadIdx.x == 0 && atomicCAS(&p.status->code, 0, 2) == 0) p.status->where = 1;
    return;
  }
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int pairs = (p.num_q_tiles + 1) / 2;
  const int pair = blockIdx.x % pairs;
  const int bh = blockIdx.x / pairs;
  const int head = bh % p.heads_q;
  const int batch = bh / p.heads_q;
  const int kv_head = head / p.group;
  const int num_tiles = (p.seq_len + kTileN - 1) / kTileN;
  const bool has_b = (2 * pair + 1) < p.num_q_tiles;

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.q_full[s], 1);
      mbar_init(&sm.pv_done[s], 1);
      mbar_init(&sm.o_full[s], 1);
      for (int b = 0; b < 2; ++b) {
        mbar_init(&sm.s_full[s][b], 1);
        mbar_init(&sm.p_full[s][b], 128);
      }
    }
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&sm.kv_full[s], 1);
      mbar_init(&sm.kv_empty[s], 2);   // one arrival per stream
    }
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 9) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 8) {
    // =============================== TMA producer =======================================
    if (elect_one_sync()) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      for (int s = 0; s < (has_b ? 2 : 1); ++s) {
        mbar_expect_tx(&sm.q_full[s], kTileM * kHeadDim * 2);
        tma_load_4d(sm.q[s][0], &tm_q, &sm.q_full[s], 0, (2 * pair + s) * kTileM, head, batch);
        tma_load_4d(sm.q[s][1], &tm_q, &sm.q_full[s], 64, (2 * pair + s) * kTileM, head, batch);
      }
    }
    __syncwarp();
    bool ok = true;
    for (int i = 0; ok && i < 2 * num_tiles; ++i) {
      const int slot = i % kSlots;
      if (i >= kSlots) {
        ok = mbar_wait(&sm.kv_empty[slot], ((i / kSlots) - 1) & 1, &sm.abort_flag, p.status, 10);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (elect_one_sync()) {
        mbar_expect_tx(&sm.kv_full[slot], kTileN * kHeadDim * 2);
        const CUtensorMap* tm = (i & 1) == 0 ? &tm_k : &tm_v;
        const int row0 = (i >> 1) * kTileN;
        tma_load_4d(sm.kv[slot][0], tm, &sm.kv_full[slot], 0, row0, kv_head, batch);
        tma_load_4d(sm.kv[slot][1], tm, &sm.kv_full[slot], 64, row0, kv_head, batch);
      }
      __syncwarp();
    }
  } else if (warp == 9 || warp == 10) {
    // =============================== UMMA issuer of stream s ============================
    const int s = warp - 9;
    if (s == 1 && !has_b) {
      // no second query tile: keep releasing the ring slots in order so that the producer advances
      bool ok = true;
      for (int i = 0; ok && i < 2 * num_tiles; ++i) {
        const int slot = i % kSlots;
        ok = mbar_wait(&sm.kv_full[slot], (i / kSlots) & 1, &sm.abort_flag, p.status, 26);
        ok = __all_sync(0xffffffffu, ok);
        if (ok && elect_one_sync()) mbar_arrive(&sm.kv_empty[slot]);
        __syncwarp();
      }
    } else {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(kTileM, kTileN, false, false);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(kTileM, kHeadDim, false, true);
      constexpr uint32_t hi_desc = umma_desc_hi_sw128(1024);
      const uint32_t q_lo0 = umma_desc_lo(smem_u32(sm.q[s][0]), 16);
      const uint32_t kv_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), 16);
      const uint32_t v_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), kTileN * 128);
      constexpr uint32_t q_half_step = (kTileM * 64 * 2) >> 4;
      constexpr uint32_t slot_step = (2 * kTileN * 64 * 2) >> 4;
      constexpr uint32_t half_step = (kTileN * 64 * 2) >> 4;
      const uint32_t tS0 = tmem + s * 128;
      const uint32_t tO = tmem + 256 + s * 128;
      auto issue_qk = [&](int t) -> bool {
        const int i = 2 * t;
        const int slot = i % kSlots;
        bool got = mbar_wait(&sm.kv_full[slot], (i / kSlots) & 1, &sm.abort_flag, p.status, 21);
        got = __all_sync(0xffffffffu, got);
        if (!got) return false;
        tc_fence_after();
        if (elect_one_sync()) {
          const uint32_t k_lo = kv_lo0 + slot * slot_step;
          const uint32_t tS = tS0 + (t & 1) * kTileN;
          umma_ss_words<false>(tS, q_lo0, hi_desc, k_lo, hi_desc, idesc_qk);
#pragma unroll
          for (int kk = 1; kk < kHeadDim / 16; ++kk) {
            umma_ss_words<true>(tS, q_lo0 + (kk >> 2) * q_half_step + (kk & 3) * 2, hi_desc,
                                k_lo + (kk >> 2) * half_step + (kk & 3) * 2, hi_desc, idesc_qk);
          }
          umma_commit(&sm.kv_empty[slot]);
          umma_commit(&sm.s_full[s][t & 1]);
        }
        __syncwarp();
        return true;
      };
      bool ok = mbar_wait(&sm.q_full[s], 0, &sm.abort_flag, p.status, 20);
      ok = __all_sync(0xffffffffu, ok);
      ok = ok && issue_qk(0);
      for (int t = 0; ok && t < num_tiles; ++t) {
        if (t + 1 < num_tiles && !issue_qk(t + 1)) break;
        const int i = 2 * t + 1;
        const int slot = i % kSlots;
        ok = mbar_wait(&sm.p_full[s][t & 1], (t >> 1) & 1, &sm.abort_flag, p.status, 22);
        ok = ok && mbar_wait(&sm.kv_full[slot], (i / kSlots) & 1, &sm.abort_flag, p.status, 23);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (elect_one_sync()) {
          const uint32_t v_lo = v_lo0 + slot * slot_step;
          const uint32_t tP = tS0 + (t & 1) * kTileN;
          umma_ts_words(tO, tP, v_lo, hi_desc, idesc_pv, t > 0 ? 1u : 0u);
#pragma unroll
          for (int kk = 1; kk < kTileN / 16; ++kk)
            umma_ts_words(tO, tP + kk * 8, v_lo + kk * 128, hi_desc, idesc_pv, 1u);
          umma_commit(&sm.kv_empty[slot]);
          umma_commit(&sm.pv_done[s]);
          if (t == num_tiles - 1) umma_commit(&sm.o_full[s]);
        }
        __syncwarp();
      }
    }
  } else {
    // =============================== softmax / epilogue of stream s =====================
    const int s = warp >> 2;
    const int row_t = tid & 127;
    if (s == 0 || has_b) {
      const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
      const uint32_t tS0 = tmem + s * 128;
      const uint32_t tO = tmem + 256 + s * 128;
      const float scale_log2 = p.scale_log2;
      const int q_row0 = (2 * pair + s) * kTileM;
      float m_used = -INFINITY;
      float l = 0.f;
      bool ok = true;
      for (int t = 0; t < num_tiles; ++t) {
        if (!mbar_wait(&sm.s_full[s][t & 1], (t >> 1) & 1, &sm.abort_flag, p.status, 30)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t tS = tS0 + (t & 1) * kTileN + lane_base;
        uint32_t r0[32], r1[32];
        tmem_ld32(tS, r0);
        tmem_ld32(tS + 32, r1);
        tmem_wait_ld();
        const int valid_cols = p.seq_len - t * kTileN;
        if (valid_cols < kTileN) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (j >= valid_cols) r0[j] = 0xff800000u;
            if (32 + j >= valid_cols) r1[j] = 0xff800000u;
          }
        }
        uint32_t pk[32];
        float sum;
        {
          const float2 sc = make_float2(scale_log2, scale_log2);
          const float2 nm = make_float2(-m_used, -m_used);
          float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(r0[2 * j]), __uint_as_float(r0[2 * j + 1])), sc, nm);
            const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(r1[2 * j]), __uint_as_float(r1[2 * j + 1])), sc, nm);
            const float2 e0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y));
            const float2 e1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
            acc0 = __fadd2_rn(acc0, e0);
            acc1 = __fadd2_rn(acc1, e1);
            pk[j] = pack_bf16x2(e0.x, e0.y);
            pk[16 + j] = pack_bf16x2(e1.x, e1.y);
          }
          sum = (acc0.x + acc0.y) + (acc1.x + acc1.y);
        }
        const bool trigger = !(sum <= 256.0f);
        if (__any_sync(0xffffffffu, trigger)) {
          float mx = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; ++j) mx = fmaxf(mx, fmaxf(__uint_as_float(r0[j]), __uint_as_float(r1[j])));
          const float m_tile = mx * scale_log2;
          float alpha = 1.f;
          if (m_tile > m_used) {
            alpha = fast_exp2(m_used - m_tile);
            m_used = m_tile;
            l *= alpha;
          }
          sum = 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(r0[2 * j]), scale_log2, -m_used));
            const float p1 = fast_exp2(fmaf(__uint_as_float(r0[2 * j + 1]), scale_log2, -m_used));
            sum += p0; sum += p1;
            pk[j] = pack_bf16x2(p0, p1);
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(r1[2 * j]), scale_log2, -m_used));
            const float p1 = fast_exp2(fmaf(__uint_as_float(r1[2 * j + 1]), scale_log2, -m_used));
            sum += p0; sum += p1;
            pk[16 + j] = pack_bf16x2(p0, p1);
          }
          if (t > 0) {
            if (!mbar_wait(&sm.pv_done[s], (t - 1) & 1, &sm.abort_flag, p.status, 32)) {
              ok = false;
              break;
            }
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < kHeadDim / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(tO + lane_base + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
              tmem_st32(tO + lane_base + c * 32, o);
            }
          }
        }
        l += sum;
        if (p.tile_lse != nullptr) {
          // [bh][query tile][key tile][row in tile]: a stream's writes are consecutive 512-byte pieces
          const int64_t qt = static_cast<int64_t>(bh) * p.num_q_tiles + (2 * pair + s);
          if (q_row0 + row_t < p.seq_len)
            __stcs(p.tile_lse + (qt * num_tiles + t) * kTileM + row_t, m_used + __log2f(sum));
        }
        tmem_st32(tS, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_full[s][t & 1]);
      }
      if (ok) ok = mbar_wait(&sm.o_full[s], 0, &sm.abort_flag, p.status, 31);
      tc_fence_after();
      const int row = q_row0 + row_t;
      const bool row_valid = row < p.seq_len;
      const float inv_l = 1.f / l;
      __nv_bfloat16* o_row = reinterpret_cast<__nv_bfloat16*>(p.o) + batch * p.o_stride_b + head * p.o_stride_h +
                             static_cast<int64_t>(row) * p.o_stride_t;
#pragma unroll
      for (int c = 0; c < kHeadDim / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tO + lane_base + c * 32, r);
        tmem_wait_ld();
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
      if (p.lse != nullptr && row_valid)
        p.lse[static_cast<int64_t>(bh) * p.seq_len + row] = (m_used + log2f(l)) * 0.69314718055994531f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

inline cudaError_t launch_pair(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                               int batch, cudaStream_t stream) {
  const int smem = static_cast<int>(sizeof(PairSmem));
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(attn_dense_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const long long ctas = static_cast<long long>(batch) * p.heads_q * ((p.num_q_tiles + 1) / 2);
  if (ctas <= 0) return cudaSuccess;
  attn_dense_pair_kernel<<<static_cast<unsigned>(ctas), kThreads, smem, stream>>>(tq, tk, tv, p);
  return cudaGetLastError();
}


}  // namespace

// Tensor maps: Q box 64 x 128 rows, K and V boxes 64 x 64 rows.
cudaError_t launch_attn_dense(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                              const AttnParams& p, int batch, cudaStream_t stream) {
  return launch_pair(tq, tk, tv, p, batch, stream);
}

}  // namespace sparsed
