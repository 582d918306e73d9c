// Dense bidirectional attention (Eq. 1 times V; the full-attention branch of Algorithm 1) for head_dim 128
// with the tensor-core instructions spanning a PAIR of CTAs on neighbouring SMs (tcgen05 cta_group::2).
//
// Why a pair: with 64-key tiles, S = Q K^T from shared memory holds the tensor pipe for the time it takes
// to read Q (128 rows) and K (64 rows) out of shared memory, 1.5 times its math time. As one M = 256 MMA
// over two SMs, each SM still reads its own 128 rows of Q but only HALF of the K tile (32 keys), and for
// O += P V only half of V (64 of the 128 head_dim columns); each SM also fetches only those halves from L2.
//
// A cluster of two CTAs owns 512 consecutive query rows of one (batch, head), as two independent
// STREAMS of 256 rows (128 per CTA). Per stream and CTA the pipeline is the one of attention.cu:
//   a producer warp   - TMA: its 128 rows of Q once, then per 64-key tile its half of K and its half of V
//                       into a ring of 8 KB slots; completion bytes of BOTH CTAs are counted on the
//                       leader CTA's barrier of the slot
//   an issuer warp    - leader CTA only: S_j = Q K_j^T (M256 N64) into one of two S buffers, then
//                       O += P_j V_j (M256 N128, P read from tensor memory); one commit per batch, delivered
//                       to the slot's barrier in both CTAs, which tells the softmax warps "S_j is ready" /
//                       "P_j V_j has drained" and the producers "the slot is free"
//   four softmax warps- one thread per query row (softmax_pipeline.cuh); each warp reports "P_j is in tensor
//                       memory" to the leader's barrier with one arrival
// so a CTA runs 12 warps (two streams) on one SM with all 512 tensor-memory columns: the same load per SM as
// two co-resident CTAs of the single-CTA kernel, without two clusters competing for one SM pair's
// tensor-memory allocator.
//
// Every wait is bounded (sm100_primitives.cuh); a CTA that gives up leaves through the cluster-wide
// tear-down barrier, and so does its peer once its own waits run out.
#include <type_traits>

#include "internal.h"
#include "sm100_pair_primitives.cuh"
#include "softmax_pipeline.cuh"

namespace sparsed {
namespace {

constexpr int kHeadDim = 128;
constexpr int kTileM = 128;        // query rows per CTA and stream
constexpr int kTileN = 64;         // keys per pipeline step
constexpr int kStreams = 2;
constexpr int kSlots = 20;         // 8 KB ring slots (half a K tile or half a V tile each), shared by both streams
constexpr int kThreads = 384;      // warps 0-3 / 4-7: softmax of stream 0 / 1; 8, 9: producers; 10, 11: issuers
constexpr int kTmemCols = 512;     // per stream 256: two S buffers of 64 columns, then O (128)
constexpr int kColS = 0;
constexpr int kColO = 128;
constexpr int kArrivalsP = 8;      // four softmax warps in each CTA of the pair

struct PairStream {
  alignas(1024) __nv_bfloat16 q[2][kTileM * 64];      // two 64-wide halves of head_dim
  uint64_t q_full;                    // used in the leader CTA: bytes of both CTAs
  uint64_t done[kSlots];              // in both CTAs: this stream's MMAs that read the slot have completed
  uint64_t p_full[2];                 // used in the leader CTA: P of both CTAs is in tensor memory
};

struct PairSmem {
  // K half-tile: two [32 keys x 64] halves of head_dim (4 KB each); V half-tile: [64 keys x 64 columns of head_dim].
  // Both streams (neighbouring query tiles of one head) read every tile from the same slot.
  alignas(1024) __nv_bfloat16 kv[kSlots][kTileN * 64];
  PairStream stream[kStreams];
  uint64_t kv_full[kSlots];           // used in the leader CTA: bytes of both CTAs
  uint32_t tmem_base;
  int abort_flag;
};

constexpr uint32_t kHi = umma_desc_hi_sw128(1024);
constexpr uint32_t kIdescQK = umma_idesc_bf16(256, 64, false, false);    // S = Q K^T, both K-major
constexpr uint32_t kIdescPV = umma_idesc_bf16(256, 128, false, true);    // O += P V, V MN-major
constexpr uint32_t kQHalfStep = (kTileM * 64 * 2) >> 4;                  // 16 KB per head_dim half of Q
constexpr uint32_t kKHalfStep = (32 * 64 * 2) >> 4;                      // 4 KB per head_dim half of a K half-tile
constexpr uint32_t kSlotStep = (kTileN * 64 * 2) >> 4;                   // 8 KB per ring slot

// kStatKeys: 0, or record one row statistic per 32 / 64 / 128 keys.
template <int kStatKeys>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_dense_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                       const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  PairSmem& sm = *reinterpret_cast<PairSmem*>(smem_raw);
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const uint32_t rank = cluster_cta_rank();   // 0 = leader
  // both CTAs of a pair see the same alignment (same kernel, same shared-memory layout), so this exit is taken
  // by both or by neither
  if ((smem_u32(smem_raw) & 1023u) != 0u) {
    if (tid == 0 && atomicCAS(&p.status->code, 0, 2) == 0) p.status->where = 3;
    return;
  }

  // ---- which rows ---------------------------------------------------------------------------
  // cluster c of a (batch, head) owns query tiles 4c .. 4c+3: stream s of CTA r has tile 4c + 2s + r
  const int cluster_id = blockIdx.x >> 1;
  const int clusters_per_head = (p.num_q_tiles + 3) >> 2;
  const int bh = cluster_id / clusters_per_head;
  const int first_tile = (cluster_id % clusters_per_head) * 4;
  const int head = bh % p.heads_q;
  const int batch = bh / p.heads_q;
  const int kv_head = head / p.group;
  const int num_tiles = (p.seq_len + kTileN - 1) / kTileN;

  // ---- set-up -------------------------------------------------------------------------------
  if (tid == 0) {
    for (int s = 0; s < kStreams; ++s) {
      PairStream& S = sm.stream[s];
      mbar_init(&S.q_full, 1);
      for (int i = 0; i < kSlots; ++i) mbar_init(&S.done[i], 1);
      mbar_init(&S.p_full[0], kArrivalsP);
      mbar_init(&S.p_full[1], kArrivalsP);
    }
    for (int i = 0; i < kSlots; ++i) mbar_init(&sm.kv_full[i], 1);
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8 && elect_one_sync()) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_o);
  }
  if (warp == 10) {
    tmem_alloc_pair(&sm.tmem_base, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  // the peer's barriers must exist before anything is signalled on them
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  bool pair_ok = true;
  {
    // the pair's instructions address both tensor memories with one base: never expected to differ
    const uint32_t peer_base = ld_cluster_u32(map_to_cta(smem_u32(&sm.tmem_base), rank ^ 1u));
    if (peer_base != tmem) {
      pair_ok = false;
      if (tid == 0 && atomicCAS(&p.status->code, 0, 4) == 0) p.status->where = 1;
    }
  }

  const int s_of_warp = warp < 8 ? (warp >> 2) : ((warp - 8) & 1);   // stream this warp serves
  PairStream& S = sm.stream[s_of_warp];
  const int q_tile = first_tile + 2 * s_of_warp + static_cast<int>(rank);
  const int q_row0 = q_tile * kTileM;
  // a stream whose leader tile lies beyond the sequence has no rows at all; one whose peer tile does still runs
  // as a pair: the peer's Q arrives as zeros and its rows are not stored
  const bool active = pair_ok && (first_tile + 2 * s_of_warp) < p.num_q_tiles;
  const uint32_t tS0 = tmem + s_of_warp * 256 + kColS;
  const uint32_t tO = tmem + s_of_warp * 256 + kColO;

  if (!active) {
    // nothing to do for this warp
  } else if (warp == 9) {
    // (spare warp)
  } else if (warp == 8) {
    // =============================== TMA producer (both streams) =============================
    const bool two = pair_ok && (first_tile + 2) < p.num_q_tiles;   // stream 1 has rows
    if (elect_one_sync()) {
      for (int s = 0; s < (two ? 2 : 1); ++s) {
        PairStream& T = sm.stream[s];
        const uint32_t q_full_leader = map_to_cta(smem_u32(&T.q_full), 0);
        const int row0 = (first_tile + 2 * s + static_cast<int>(rank)) * kTileM;
        if (rank == 0) mbar_expect_tx(&T.q_full, 2 * kTileM * kHeadDim * 2);   // rows beyond the sequence arrive as zeros
        tma_load_4d_pair(T.q[0], &tm_q, q_full_leader, 0, row0, head, batch);
        tma_load_4d_pair(T.q[1], &tm_q, q_full_leader, 64, row0, head, batch);
      }
    }
    __syncwarp();
    bool ok = true;
    // load i: this CTA's half of K (even) or V (odd) of tile i / 2, for both streams
    for (int i = 0; ok && i < 2 * num_tiles; ++i) {
      const int slot = i % kSlots;
      if (i >= kSlots) {
        // free once the MMAs of every stream that read it have completed
        const uint32_t parity = ((i / kSlots) - 1) & 1;
        ok = two ? mbar_wait2(&sm.stream[0].done[slot], parity, &sm.stream[1].done[slot], parity, &sm.abort_flag,
                              p.status, 40)
                 : mbar_wait(&sm.stream[0].done[slot], parity, &sm.abort_flag, p.status, 40);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (elect_one_sync()) {
        const uint32_t full_leader = map_to_cta(smem_u32(&sm.kv_full[slot]), 0);
        if (rank == 0) mbar_expect_tx(&sm.kv_full[slot], 2 * kTileN * 64 * 2);   // both CTAs' halves
        const int key0 = (i >> 1) * kTileN;
        if ((i & 1) == 0) {
          // keys [32 rank, 32 rank + 32) of the tile, all of head_dim
          tma_load_4d_pair(sm.kv[slot], &tm_k, full_leader, 0, key0 + 32 * static_cast<int>(rank), kv_head, batch);
          tma_load_4d_pair(sm.kv[slot] + 32 * 64, &tm_k, full_leader, 64, key0 + 32 * static_cast<int>(rank), kv_head,
                           batch);
        } else {
          // all 64 keys, head_dim columns [64 rank, 64 rank + 64)
          tma_load_4d_pair(sm.kv[slot], &tm_v, full_leader, 64 * static_cast<int>(rank), key0, kv_head, batch);
        }
      }
      __syncwarp();
    }
  } else if (warp == 10 || warp == 11) {
    // =============================== UMMA issuer (leader CTA) ================================
    if (rank == 0) {
      const uint32_t q_lo0 = umma_desc_lo(smem_u32(S.q[0]), 16);
      const uint32_t k_lo0 = umma_desc_lo(smem_u32(sm.kv[0]), 16);             // as K (K-major)
      const uint32_t v_lo0 = umma_desc_lo(smem_u32(sm.kv[0]), kTileN * 128);   // as V (MN-major, one 64-wide atom)
      bool ok = true;
      // S_t = Q K_t^T into S buffer t & 1: eight M256 N64 K16 MMAs
      auto issue_qk = [&](int t) -> bool {
        const int g = 2 * t;
        const int slot = g % kSlots;
        bool got = mbar_wait(&sm.kv_full[slot], (g / kSlots) & 1, &sm.abort_flag, p.status, 41);
        got = __all_sync(0xffffffffu, got);
        if (!got) return false;
        tc_fence_after();
        if (elect_one_sync()) {
          const uint32_t d = tS0 + (t & 1) * kTileN;
          const uint32_t k_lo = k_lo0 + slot * kSlotStep;
          umma_ss_pair<false>(d, q_lo0, kHi, k_lo, kHi, kIdescQK);
#pragma unroll
          for (int kk = 1; kk < 8; ++kk)
            umma_ss_pair<true>(d, q_lo0 + (kk >> 2) * kQHalfStep + (kk & 3) * 2, kHi,
                               k_lo + (kk >> 2) * kKHalfStep + (kk & 3) * 2, kHi, kIdescQK);
          umma_commit_pair(&S.done[slot]);
        }
        __syncwarp();
        return true;
      };
      ok = mbar_wait(&S.q_full, 0, &sm.abort_flag, p.status, 42);
      ok = __all_sync(0xffffffffu, ok);
      ok = ok && issue_qk(0);
      for (int t = 0; ok && t < num_tiles; ++t) {
        // The S buffer of tile t+1 last held P of tile t-1, whose P V was issued earlier by this thread, and
        // tcgen05 operations of one thread execute in issue order.
        if (t + 1 < num_tiles && !issue_qk(t + 1)) {
          ok = false;
          break;
        }
        const int g = 2 * t + 1;
        const int slot = g % kSlots;
        ok = mbar_wait2(&S.p_full[t & 1], (t >> 1) & 1, &sm.kv_full[slot], (g / kSlots) & 1, &sm.abort_flag, p.status,
                        43);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (elect_one_sync()) {
          // O (+)= P_t V_t: four M256 N128 K16 MMAs, 16 keys (2048 bytes of V) per step
          const uint32_t a = tS0 + (t & 1) * kTileN;
          const uint32_t v_lo = v_lo0 + slot * kSlotStep;
          umma_ts_pair(tO, a, v_lo, kHi, kIdescPV, t > 0 ? 1u : 0u);
#pragma unroll
          for (int kk = 1; kk < 4; ++kk) umma_ts_pair(tO, a + kk * 8, v_lo + kk * 128, kHi, kIdescPV, 1u);
          umma_commit_pair(&S.done[slot]);
        }
        __syncwarp();
      }
    }
  } else {
    // =============================== softmax / epilogue ======================================
    const int row_in_tile = tid & (kTileM - 1);
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const float scale_log2 = p.scale_log2;
    const uint32_t p_full_leader0 = map_to_cta(smem_u32(&S.p_full[0]), 0);
    const uint32_t p_full_leader1 = map_to_cta(smem_u32(&S.p_full[1]), 0);
    bool ok = true;
    RowState st{-INFINITY, 0.f};
    RowStatWriter<kStatKeys> stats;
    if constexpr (kStatKeys > 0) {
      const int groups = (p.seq_len + kStatKeys - 1) / kStatKeys;
      float* first = nullptr;
      if (p.tile_lse != nullptr && q_row0 + row_in_tile < p.seq_len)
        first = p.tile_lse + (static_cast<int64_t>(bh) * p.num_q_tiles + q_tile) * groups * kTileM + row_in_tile;
      stats.init(first, groups);
    }
    // One 64-key tile of the softmax; kOdd (a compile-time tag) is used by the walk that records one statistic per
    // 128 keys, which runs its tiles in pairs.
    auto tile_body = [&](int t, auto odd_tag) -> bool {
      [[maybe_unused]] constexpr bool kOdd = decltype(odd_tag)::value;
      // S_t is ready when the Q K^T batch that read ring load 2t has completed
      const int gk = 2 * t;
      if (!mbar_wait(&S.done[gk % kSlots], (gk / kSlots) & 1, &sm.abort_flag, p.status, 44)) return false;
      tc_fence_after();
      const int buf = t & 1;
      const uint32_t tS = tS0 + buf * kTileN + lane_base;
      uint32_t pk[32];
      uint32_t r0[32], r1[32];
      tmem_ld32(tS, r0);
      tmem_ld32(tS + 32, r1);
      tmem_wait_ld();
      const int valid_cols = p.seq_len - t * kTileN;   // ragged tail of the sequence
      if (valid_cols < kTileN) mask_columns_from(r0, r1, valid_cols);
      float2 sums;
      bool exact = (st.m == -INFINITY);   // nothing accumulated yet: no reference maximum to try
      if (!__all_sync(0xffffffffu, exact)) {
        sums = softmax_group_fast(r0, r1, scale_log2, st.m, pk);
        exact = !(sums.x + sums.y <= 256.0f);   // logits outgrew the running maximum (or NaN)
      }
      if (__any_sync(0xffffffffu, exact)) {
        const float alpha = softmax_group_exact(r0, r1, scale_log2, st, pk, sums);
        if constexpr (kStatKeys > 0) stats.rescale(alpha);
        if (t > 0) {
          // O must be quiescent: wait until P_{t-1} V_{t-1} (which read ring load 2t-1) has drained
          const int gp = 2 * (t - 1) + 1;
          if (!mbar_wait(&S.done[gp % kSlots], (gp / kSlots) & 1, &sm.abort_flag, p.status, 45)) return false;
          tc_fence_after();
          rescale_accumulator_row(tO + lane_base, alpha);
          if (p.slow_path_events != nullptr && lane == 0) atomicAdd(p.slow_path_events, 1ull);
        }
      }
      st.l += sums.x + sums.y;
      if constexpr (kStatKeys > 0) stats.begin(sums, kOdd);
      tmem_st32(tS, pk);  // P_t over the first 32 columns of S_t
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(buf ? p_full_leader1 : p_full_leader0);
      // the statistic is stored after P has been handed over: off the S -> P -> P V chain
      if constexpr (kStatKeys > 0) stats.finish(st.m, kOdd);
      return true;
    };
    {
      int t = 0;
      for (; ok && t + 1 < num_tiles; t += 2) ok = tile_body(t, std::false_type{}) && tile_body(t + 1, std::true_type{});
      if (ok && t < num_tiles) ok = tile_body(t, std::false_type{});
    }
    // ---- epilogue: O / l -> bf16 -> shared memory -> global -----------------------------------
    // Every thread goes through the barrier below even after a wait has run out (it then stages zeros), so that
    // none is left waiting there; what is done after it is decided by the shared flag.
    if (ok) {
      const int gl = 2 * (num_tiles - 1) + 1;   // the last P V read this load's slot
      ok = mbar_wait(&S.done[gl % kSlots], (gl / kSlots) & 1, &sm.abort_flag, p.status, 46);
    }
    tc_fence_after();
    const int row = q_row0 + row_in_tile;
    const float inv_l = st.l > 0.f ? (1.f / st.l) : 0.f;
    // the stream's Q tile is dead (its last Q K^T completed before its last P V did): it stages the output tile
    stage_output_row(tO + lane_base, ok, inv_l, &S.q[0][0], row_in_tile);
    named_barrier_sync(1 + s_of_warp, kTileM);
    if (*reinterpret_cast<volatile int*>(&sm.abort_flag) == 0) {
      if (row_in_tile == 0 && q_row0 < p.seq_len) {
        // rows beyond the sequence end are clipped by the tensor map
        tma_store_4d(&tm_o, S.q[0], 0, q_row0, head, batch);
        tma_store_4d(&tm_o, S.q[1], 64, q_row0, head, batch);
        tma_store_commit();
        tma_store_wait_read();
      }
      if (p.lse != nullptr && row < p.seq_len)
        p.lse[static_cast<int64_t>(bh) * p.seq_len + row] = (st.m + log2f(st.l)) * 0.69314718055994531f;
    }
  }

  // ---- teardown -------------------------------------------------------------------------------
  // neither CTA may leave (or free its tensor memory) while the pair's MMAs, loads or arrivals can still touch it
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == 10) {
    __syncwarp();
    tmem_dealloc_pair(tmem, kTmemCols);
  }
}

template <int kStatKeys>
cudaError_t launch_pair(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                        const AttnParams& p, cudaStream_t stream) {
  auto kernel = attn_dense_pair_kernel<kStatKeys>;
  const int smem = static_cast<int>(sizeof(PairSmem));
  static SmemLimit limit;  // per template instantiation
  cudaError_t e = ensure_dynamic_smem(kernel, smem, limit);
  if (e != cudaSuccess) return e;
  const long long bh = p.num_q_tiles > 0 ? p.num_items / p.num_q_tiles : 0;
  const long long clusters = bh * ((p.num_q_tiles + 3) / 4);
  if (clusters <= 0) return cudaSuccess;
  kernel<<<static_cast<unsigned>(2 * clusters), kThreads, smem, stream>>>(tq, tk, tv, to, p);
  return cudaGetLastError();
}

}  // namespace

// Tensor maps: Q and O boxes 64 x 128 rows, K box 64 x 32 rows, V box 64 x 64 rows. p.num_q_tiles = ceil(seq_len / 128).
cudaError_t launch_attn_dense_pair(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                   const CUtensorMap& to, const AttnParams& p, cudaStream_t stream) {
  if (p.tile_lse == nullptr) return launch_pair<0>(tq, tk, tv, to, p, stream);
  if (p.stat_keys == 128) return launch_pair<128>(tq, tk, tv, to, p, stream);
  if (p.stat_keys == 64) return launch_pair<64>(tq, tk, tv, to, p, stream);
  return launch_pair<32>(tq, tk, tv, to, p, stream);
}

}  // namespace sparsed
