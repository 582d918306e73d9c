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
//                 is issued before P_t V_t. Each batch of MMAs ends in one commit to the stream's
//                 barrier for the ring slot it read; the softmax warps wait on it for "S_t ready" /
//                 "P_t V_t drained", and the producer reuses a slot once both streams' barriers for
//                 it have completed (one commit per batch: the issuing thread is the bottleneck).
//   warps 0-3, 4-7 : softmax warpgroup of stream 0 / 1, one thread per query row: the same
//                 single-pass online softmax with a stale running maximum as in the sparse kernel.
// The streams share nothing else (own S buffers, O accumulator, maxima), so they drift apart and
// one stream's softmax overlaps the other's MMAs. Tensor memory: 2 x (2 x 64 S + 128 O) = 512
// columns; shared memory 208 KB. Optional outputs: LSE, and the per-(row, 64-key tile) statistic
// m + log2(sum p) from which the switch step's pooled scores are formed (laid out
// [batch*head][128-row query tile][key tile][row], so that both this kernel's writes and the
// pooling kernel's reads are contiguous per query tile).
#include "internal.h"
#include "softmax_pipeline.cuh"

namespace sparsed {
namespace {


constexpr int kHeadDim = 128;
constexpr int kTileM = 128;
constexpr int kTileN = 64;
constexpr int kSlots = 9;             // 16 KB each, shared by K and V: load 2t is K_t, load 2t+1 is V_t
constexpr int kThreads = 352;         // warps 0-3 softmax A, 4-7 softmax B, 8 TMA, 9 UMMA A, 10 UMMA B
constexpr int kTmemCols = 512;
#ifndef SPARSED_ATTN_POLY_EVERY
#define SPARSED_ATTN_POLY_EVERY 0
#endif
constexpr int kPolyEvery = SPARSED_ATTN_POLY_EVERY;  // every n-th exponential on the FMA pipes (0 = none)

struct PairSmem {
  alignas(1024) __nv_bfloat16 q[2][2][kTileM * 64];
  alignas(1024) __nv_bfloat16 kv[kSlots][2][kTileN * 64];
  uint64_t q_full[2], kv_full[kSlots];
  uint64_t done[2][kSlots];   // [stream][slot]: the stream's MMAs that read the slot have completed
  uint64_t p_full[2][2];
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
#ifdef SPARSED_TIMELINE
  // debug: SM clock during the kernel = clock64 ticks per globaltimer nanosecond, seen by one CTA
  long long tl_c0 = 0, tl_g0 = 0;
  if (blockIdx.x == 700 && tid == 0) {
    tl_c0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tl_g0));
  }
#endif
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
      for (int b = 0; b < 2; ++b) mbar_init(&sm.p_full[s][b], 128);
      for (int b = 0; b < kSlots; ++b) mbar_init(&sm.done[s][b], 1);
    }
    for (int s = 0; s < kSlots; ++s) mbar_init(&sm.kv_full[s], 1);
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
        // the slot's previous occupant has been read by both streams
        const uint32_t parity = ((i / kSlots) - 1) & 1;
        ok = has_b ? mbar_wait2(&sm.done[0][slot], parity, &sm.done[1][slot], parity, &sm.abort_flag, p.status, 10)
                   : mbar_wait(&sm.done[0][slot], parity, &sm.abort_flag, p.status, 10);
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
    if (s == 0 || has_b) {
      const uint32_t q_lo0 = umma_desc_lo(smem_u32(sm.q[s][0]), 16);
      const uint32_t kv_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), 16);
      const uint32_t v_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), kTileN * 128);
      constexpr uint32_t slot_step = (2 * kTileN * 64 * 2) >> 4;
      const uint32_t tS0 = tmem + s * 128;
      const uint32_t tO = tmem + 256 + s * 128;
      auto issue_qk = [&](int t) -> bool {
        const int i = 2 * t;
        const int slot = i % kSlots;
        bool got = mbar_wait(&sm.kv_full[slot], (i / kSlots) & 1, &sm.abort_flag, p.status, 21);
        got = __all_sync(0xffffffffu, got);
        if (!got) return false;
        issue_qk64(tS0 + (t & 1) * kTileN, q_lo0, kv_lo0 + slot * slot_step, &sm.done[s][slot]);
        return true;
      };
      bool ok = mbar_wait(&sm.q_full[s], 0, &sm.abort_flag, p.status, 20);
      ok = __all_sync(0xffffffffu, ok);
      ok = ok && issue_qk(0);
      for (int t = 0; ok && t < num_tiles; ++t) {
        if (t + 1 < num_tiles && !issue_qk(t + 1)) break;
        const int i = 2 * t + 1;
        const int slot = i % kSlots;
        ok = mbar_wait2(&sm.p_full[s][t & 1], (t >> 1) & 1, &sm.kv_full[slot], (i / kSlots) & 1, &sm.abort_flag,
                        p.status, 22);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        issue_pv64(tO, tS0 + (t & 1) * kTileN, v_lo0 + slot * slot_step, t > 0, &sm.done[s][slot]);
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
      RowState st{-INFINITY, 0.f};
      RowStatWriter stats;
      {
        const int groups = (p.seq_len + p.stat_keys - 1) / p.stat_keys;
        float* first = nullptr;
        if (p.tile_lse != nullptr && q_row0 + row_t < p.seq_len)
          first = p.tile_lse + (static_cast<int64_t>(bh) * p.num_q_tiles + (2 * pair + s)) * groups * kTileM + row_t;
        stats.init(first, p.stat_keys, groups);
      }
      bool ok = true;
      for (int t = 0; t < num_tiles; ++t) {
        // S_t is ready when this stream's Q K^T batch that read ring slot 2t has completed
        if (!mbar_wait(&sm.done[s][(2 * t) % kSlots], ((2 * t) / kSlots) & 1, &sm.abort_flag, p.status, 30)) {
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
        if (valid_cols < kTileN) mask_columns_from(r0, r1, valid_cols);
        uint32_t pk[32];
        float2 sums = softmax_group_fast<kPolyEvery>(r0, r1, scale_log2, st.m, pk);
        const bool trigger = !(sums.x + sums.y <= 256.0f);
        if (__any_sync(0xffffffffu, trigger)) {
          const float alpha = softmax_group_exact(r0, r1, scale_log2, st, pk, sums);
          if (t > 0) {
            // O must be quiescent: wait until P_{t-1} V_{t-1} (which read ring slot 2t-1) has drained
            const int ip = 2 * (t - 1) + 1;
            if (!mbar_wait(&sm.done[s][ip % kSlots], (ip / kSlots) & 1, &sm.abort_flag, p.status, 32)) {
              ok = false;
              break;
            }
            tc_fence_after();
            rescale_accumulator_row(tO + lane_base, alpha);
            if (p.slow_path_events != nullptr && (tid & 31) == 0) atomicAdd(p.slow_path_events, 1ull);
          }
        }
        st.l += sums.x + sums.y;
        stats.put(t, sums, st.m);
        tmem_st32(tS, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_full[s][t & 1]);
      }
      if (ok) {
        const int il = 2 * (num_tiles - 1) + 1;   // the last P V read ring slot il
        ok = mbar_wait(&sm.done[s][il % kSlots], (il / kSlots) & 1, &sm.abort_flag, p.status, 31);
      }
      tc_fence_after();
      const int row = q_row0 + row_t;
      const bool row_valid = row < p.seq_len;
      const float inv_l = 1.f / st.l;
      __nv_bfloat16* o_row = reinterpret_cast<__nv_bfloat16*>(p.o) + batch * p.o_stride_b + head * p.o_stride_h +
                             static_cast<int64_t>(row) * p.o_stride_t;
      store_output_row(tO + lane_base, true, inv_l, o_row, row_valid);
      if (p.lse != nullptr && row_valid)
        p.lse[static_cast<int64_t>(bh) * p.seq_len + row] = (st.m + log2f(st.l)) * 0.69314718055994531f;
    }
  }

  tc_fence_before();
  __syncthreads();
#ifdef SPARSED_TIMELINE
  if (blockIdx.x == 700 && tid == 0) {
    long long g1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
    long long* out = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(p.status) + 64);
    out[0] = clock64() - tl_c0;
    out[1] = g1 - tl_g0;
  }
#endif
  if (warp == 9) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

inline cudaError_t launch_pair(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                               int batch, cudaStream_t stream) {
  const int smem = static_cast<int>(sizeof(PairSmem));
  static SmemLimit limit;
  cudaError_t e = ensure_dynamic_smem(attn_dense_pair_kernel, smem, limit);
  if (e != cudaSuccess) return e;
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
