// Attention for head_dim 128, bf16 in / bf16 out, fp32 softmax, on sm_100a, from one kernel:
// dense bidirectional attention (Eq. 1 times V; the full-attention branch of Algorithm 1) and
// block-sparse attention over CSR block lists (Eq. 3 / Eq. 4 times V; the "Sparse Reusing" branch).
//
// One CTA owns 128 consecutive query rows of one (batch, head) and streams 64-key tiles through a
// warp-specialised pipeline:
//   warp 4  : TMA producer  - Q once, then a K tile and a V tile per step into a ring of
//                             128B-swizzled shared memory shared by K and V
//   warp 5  : UMMA issuer   - S_j = Q K_j^T into one of two tensor-memory buffers, then
//                             O += P_j V_j with P read from tensor memory (P overwrites the
//                             first half of S_j's columns). S_{j+1} is issued before P_j V_j,
//                             so the tensor pipe works on the next logits while the softmax
//                             warps are busy with the current ones. Each batch of MMAs ends in ONE
//                             commit to the barrier of the ring slot it read: that barrier tells the
//                             softmax warps "S_j is ready" / "P_j V_j has drained" and the producer
//                             "the slot is free" (the issuing thread is the pipeline's bottleneck:
//                             a commit costs it about 150 clocks, a barrier poll about 100).
//   warps 0-3: one thread per query row - single-pass online softmax in fp32 on base-2 logits
//             against a stale running maximum (softmax_pipeline.cuh); finally O is normalised
//             and stored.
// Two CTAs fit on one SM (at most 112 KB of shared memory and 256 tensor-memory columns each).
//
// Where the keys come from:
//   * dense: every 64-key tile of the sequence in order; the last one may be ragged (any seq_len).
//     Optional output: the rows' LSE. (The dense pass that also records the row statistics of the switch
//     step runs on a kernel of its own, attention_dense_pair.cu.)
//   * 128-key blocks: the 128 query rows are one query block; its CSR list is walked as it is,
//     two tiles per block.
//   * 64- and 32-key blocks: the 128 query rows are two / four consecutive query blocks with lists
//     of their own. The CTA walks the UNION of those lists (built in shared memory at start-up as one
//     bitmap per query block) and every warp masks, per 32-column chunk of a tile, the key blocks
//     its own query block did not keep; a tile in which a warp keeps nothing costs it no
//     exponentials. All 128 rows of every MMA belong to real queries, and neighbouring query blocks
//     share the K/V tiles they have in common.
#include "internal.h"
#include "softmax_pipeline.cuh"

namespace sparsed {
namespace {

constexpr int kHeadDim = 128;
constexpr int kTileM = 128;   // UMMA M; rows of tensor memory
constexpr int kTileN = 64;    // keys per pipeline step
constexpr int kSoftmaxThreads = 128;
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;
constexpr int kColS = 0;      // two S buffers of 64 fp32 columns; P (bf16 pairs) reuses the first 32
constexpr int kColO = 128;    // O accumulator (fp32, 128 columns)
constexpr int kMaxPackedBlocks = 2048;   // key blocks per row the union walk can hold (64- and 32-key blocks)

// Debug builds (-DSPARSED_TIMELINE) record clock64 stamps of one CTA's pipeline roles after the
// workspace status block: 3 regions of 2048 int64 (softmax thread 0, UMMA thread, TMA thread).
#ifdef SPARSED_TIMELINE
#define TL_DECL(region) long long* tl_buf = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(p.status) + 1024) + (region) * 2048; int tl_n = 0; const bool tl_on = (blockIdx.x == 1000) && (threadIdx.x == 0 || threadIdx.x == 128 || threadIdx.x == 160);
#define TL(tag) do { if (tl_on && tl_n < 2047) { tl_buf[1 + tl_n++] = (static_cast<long long>(tag) << 48) | (clock64() & 0xFFFFFFFFFFFFll); tl_buf[0] = tl_n; } } while (0)
#else
#define TL_DECL(region)
#define TL(tag)
#endif

// Ring slots: five for 128-key blocks; four when the union walk needs room for its lists.
template <int kBlock>
struct AttnSmem {
  static constexpr bool kPacked = kBlock < kTileM;
  static constexpr int kSlots = kPacked ? 4 : 5;
  static constexpr int kGroups = kTileM / kBlock;                       // query blocks per CTA
  static constexpr int kWords = kPacked ? kMaxPackedBlocks / 32 : 1;    // bitmap words per query block
  alignas(1024) __nv_bfloat16 q[2][kTileM * 64];           // two 64-wide halves of head_dim
  alignas(1024) __nv_bfloat16 kv[kSlots][2][kTileN * 64];  // each slot: two 64-wide halves of head_dim
  uint64_t q_full, kv_full[kSlots];
  uint64_t done[kSlots];   // the MMAs that read the slot have completed (Q K^T for a K tile, P V for a V tile)
  uint64_t p_full[2];
  uint64_t q_free;         // an output tile has been read out of the Q buffer (which staged it): the next Q may land
  uint32_t tmem_base;
  int abort_flag;
  int n_union;                                             // packed: key blocks in the union list
  uint32_t member[kGroups][kWords];                        // packed: bit j of query block g = "g keeps key block j"
  uint16_t union_ids[kPacked ? kMaxPackedBlocks : 2];      // packed: the union, ascending
};

// kDense: walk every key tile of the sequence (kBlock must be 128 then; no block lists are read).
// kMultiItem: a CTA may be given several query tiles (launched with fewer CTAs than tiles); without it the
// item loops below run once and their running counters fold to zero at compile time.
template <int kBlock, bool kDense, bool kMultiItem>
__global__ void __launch_bounds__(kThreads, 2)
attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, const AttnParams p) {
  static_assert(!kDense || kBlock == 128, "the dense walk uses the unpacked layout");
  static_assert(!kMultiItem || kBlock == 128, "the packed walk prepares its union once per CTA");
  using Smem = AttnSmem<kBlock>;
  constexpr bool kPacked = Smem::kPacked;
  constexpr int kSlots = Smem::kSlots;
  constexpr int kGroups = Smem::kGroups;
  constexpr int kTilesPerBlock = kBlock >= kTileN ? kBlock / kTileN : 1;   // 128-key block: two tiles
  constexpr int kBlocksPerTile = kBlock >= kTileN ? 1 : kTileN / kBlock;   // 32-key blocks: two per tile
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0u) {
    // swizzled tiles need a 1024-byte aligned base; never expected, reported instead of trusted
    if (threadIdx.x == 0 && atomicCAS(&p.status->code, 0, 2) == 0) p.status->where = 1;
    return;
  }

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  // ---- work items ----------------------------------------------------------------------
  // An item is one 128-row query tile of one (batch, head). A CTA takes items blockIdx.x,
  // blockIdx.x + gridDim.x, ... ; the host launches either one CTA per item or (dense and 128-key
  // blocks only) as many CTAs as fit on the device at once, in which case each role of the pipeline
  // runs on into its next item on its own: the producer loads the next Q, list and K/V tiles while
  // the softmax warps are still in the previous item's last tiles and epilogue, so the start-up
  // chain row_ptr -> col_idx -> first K tile -> first MMA of all but a CTA's first item is hidden.
  // Every counter below (loads, tiles, Q loads) runs on across items and all roles compute the same
  // values, so ring slots, S buffers and barrier phases simply continue.
  struct Item {
    int q_tile, bh, head, batch, kv_head, q_row0, groups_here, r0;
    int list_begin, list_len;   // CSR entries of the item's query blocks; dense: key tiles of the sequence
  };
  const int n_items = p.num_items;
  auto describe = [&](int item) -> Item {
    Item it;
    it.q_tile = item % p.num_q_tiles;
    it.bh = item / p.num_q_tiles;
    it.head = it.bh % p.heads_q;
    it.batch = it.bh / p.heads_q;
    it.kv_head = it.head / p.group;
    it.q_row0 = it.q_tile * kTileM;
    const int qb0 = it.q_tile * kGroups;                                   // first query block of the item
    it.groups_here = kDense ? 1 : min(kGroups, p.num_blocks - qb0);        // the last tile of a head may hold fewer
    it.r0 = it.bh * p.num_blocks + qb0;                                    // CSR row of query block qb0
    it.list_begin = 0;
    it.list_len = (p.seq_len + kTileN - 1) / kTileN;
    if constexpr (!kDense) {
      // adjacent rows are adjacent in col_idx, so the item's lists are one run of entries
      it.list_begin = __ldg(p.row_ptr + it.r0);
      it.list_len = __ldg(p.row_ptr + it.r0 + it.groups_here) - it.list_begin;
      if (it.list_begin < 0 || it.list_len < 0 ||
          static_cast<int64_t>(it.list_begin) + it.list_len > p.col_capacity) {
        // row_ptr points outside col_idx: not followed; the rows get zeros and the status word says why
        if (atomicCAS(&p.status->code, 0, 3) == 0) p.status->where = 2;
        it.list_begin = 0;
        it.list_len = 0;
      }
    }
    return it;
  };
  // tiles of an item in the unpacked walks (the packed walk counts its union instead)
  auto unpacked_tiles = [&](const Item& it) -> int { return kDense ? it.list_len : it.list_len * kTilesPerBlock; };

  const int first_item = blockIdx.x;
  Item cur = describe(first_item);

  // ---- set-up --------------------------------------------------------------------------
  // The producer warp owns the barriers of its own loads, so it can start them before the CTA-wide
  // set-up (tensor-memory allocation, the other barriers) has finished: the Q tile, the first block
  // ids of the list and, when the list needs no preparation, the first ring-full of K/V tiles.
  int list_ids = 0;     // unpacked walk: lane i holds the block id of list entry 32 * chunk + i
  int loads_issued = 0; // K/V loads of the first item already issued by the producer before the set-up barrier
  // rows [kv_row0, +64) (or two 32-row blocks at kv_row0 / kv_row1) of K (which = 0) or V into `slot`
  auto issue_load = [&](const Item& it, int slot, int which, int kv_row0, int kv_row1, int blocks_here) {
    if (elect_one_sync()) {
      const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
      if constexpr (kBlocksPerTile == 1) {
        mbar_expect_tx(&sm.kv_full[slot], kTileN * kHeadDim * 2);
        tma_load_4d(sm.kv[slot][0], tm, &sm.kv_full[slot], 0, kv_row0, it.kv_head, it.batch);
        tma_load_4d(sm.kv[slot][1], tm, &sm.kv_full[slot], 64, kv_row0, it.kv_head, it.batch);
      } else {
        // tensor-map boxes are 32 rows here; block b of the tile lands at rows 32 b
        mbar_expect_tx(&sm.kv_full[slot], blocks_here * kBlock * kHeadDim * 2);
        tma_load_4d(sm.kv[slot][0], tm, &sm.kv_full[slot], 0, kv_row0, it.kv_head, it.batch);
        tma_load_4d(sm.kv[slot][1], tm, &sm.kv_full[slot], 64, kv_row0, it.kv_head, it.batch);
        if (blocks_here == 2) {
          tma_load_4d(sm.kv[slot][0] + kBlock * 64, tm, &sm.kv_full[slot], 0, kv_row1, it.kv_head, it.batch);
          tma_load_4d(sm.kv[slot][1] + kBlock * 64, tm, &sm.kv_full[slot], 64, kv_row1, it.kv_head, it.batch);
        }
      }
    }
    __syncwarp();
  };
  auto issue_q_load = [&](const Item& it) {
    if (elect_one_sync()) {
      mbar_expect_tx(&sm.q_full, kTileM * kHeadDim * 2);   // rows beyond the sequence arrive as zeros
      tma_load_4d(sm.q[0], &tm_q, &sm.q_full, 0, it.q_row0, it.head, it.batch);
      tma_load_4d(sm.q[1], &tm_q, &sm.q_full, 64, it.q_row0, it.head, it.batch);
    }
    __syncwarp();
  };
  // first key row of tile t in the unpacked walks
  auto unpacked_row = [&](int t) -> int {
    if constexpr (kDense) return t * kTileN;
    const int e = t / kTilesPerBlock;
    return __shfl_sync(0xffffffffu, list_ids, e & 31) * kBlock + (t % kTilesPerBlock) * kTileN;
  };
  if (warp == 4) {
    if (lane == 0) {
      mbar_init(&sm.q_full, 1);
      for (int s = 0; s < kSlots; ++s) mbar_init(&sm.kv_full[s], 1);
      mbar_fence_init();
    }
    __syncwarp();
    if (elect_one_sync()) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      if constexpr (!kDense) tma_prefetch_desc(&tm_o);
    }
    __syncwarp();
    if (cur.list_len > 0) {
      issue_q_load(cur);
      if constexpr (!kPacked) {
        if constexpr (!kDense) {
          if (lane < cur.list_len) list_ids = __ldg(p.col_idx + cur.list_begin + lane);
        }
        const int first = min(2 * unpacked_tiles(cur), kSlots);   // list entries 0..2 at most: within the first chunk
        for (; loads_issued < first; ++loads_issued)
          issue_load(cur, loads_issued, loads_issued & 1, unpacked_row(loads_issued >> 1), 0, 1);
      }
    }
  }
  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) mbar_init(&sm.done[s], 1);
    for (int s = 0; s < 2; ++s) mbar_init(&sm.p_full[s], kSoftmaxThreads);
    mbar_init(&sm.q_free, 1);
    sm.abort_flag = 0;
    sm.n_union = 0;
    mbar_fence_init();
  }
  if constexpr (kBlocksPerTile > 1) {
    // a tile may be half filled (odd union): its other half is multiplied by P = 0, so it has to
    // hold finite numbers from the start
    uint4* z = reinterpret_cast<uint4*>(&sm.kv[0][0][0]);
    constexpr int n16 = kSlots * 2 * kTileN * 64 * 2 / 16;
    for (int i = tid; i < n16; i += kThreads) z[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
  }
  if (warp == 5) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  if constexpr (kPacked) {
    // (one item per CTA here) One bitmap per query block, then their union as an ascending list.
    const int words = (p.num_blocks + 31) >> 5;
    for (int i = tid; i < kGroups * Smem::kWords; i += kThreads) (&sm.member[0][0])[i] = 0u;
    __syncthreads();
    int bound[kGroups];   // bound[g] = first CSR entry after query block g's list
#pragma unroll
    for (int g = 0; g < kGroups; ++g) bound[g] = __ldg(p.row_ptr + cur.r0 + min(g + 1, cur.groups_here));
    for (int e = cur.list_begin + tid; e < cur.list_begin + cur.list_len; e += kThreads) {
      const int id = __ldg(p.col_idx + e);
      int g = 0;
#pragma unroll
      for (int j = 0; j + 1 < kGroups; ++j) g += (e >= bound[j]) ? 1 : 0;
      if (id >= 0 && id < p.num_blocks) atomicOr(&sm.member[g][id >> 5], 1u << (id & 31));
    }
    __syncthreads();
    if (warp == 4) {
      int base = 0;
      for (int w0 = 0; w0 < words; w0 += 32) {
        const int w = w0 + lane;
        uint32_t bits = 0u;
        if (w < words) {
#pragma unroll
          for (int g = 0; g < kGroups; ++g) bits |= sm.member[g][w];
        }
        const int cnt = __popc(bits);
        int incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, off);
          if (lane >= off) incl += v;
        }
        int pos = base + incl - cnt;
        while (bits != 0u) {
          const int b = __ffs(bits) - 1;
          sm.union_ids[pos++] = static_cast<uint16_t>(w * 32 + b);
          bits &= bits - 1u;
        }
        base += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) sm.n_union = base;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tO = tmem + kColO;
  // key blocks an item walks (dense: key tiles) and its tiles
  auto entries_of = [&](const Item& it) -> int { return kPacked ? sm.n_union : it.list_len; };
  auto tiles_of = [&](const Item& it) -> int {
    const int n = entries_of(it);
    return kDense ? n : kBlocksPerTile == 1 ? n * kTilesPerBlock : (n + kBlocksPerTile - 1) / kBlocksPerTile;
  };

  // Warps 4 and 5 run their loops with all 32 lanes converged and let one elected lane issue
  // the TMA / UMMA instructions: their operands then stay on the uniform datapath.
  if (warp == 4) {
    // =============================== TMA producer =======================================
    TL_DECL(2)
    bool ok = true;
    int load0 = 0;       // K/V loads issued for earlier items
    int q_tiles_done = 0;  // earlier items that had keys (each loaded a Q tile and staged an output tile)
    for (int item = first_item; ok && item < n_items; item += gridDim.x) {
      // The Q buffer doubles as the staging tile of the previous output: the next Q may land once the softmax
      // warps have had that output read out of it (which is after the item's last MMA). The first ring-full of
      // the new item's K/V loads does not depend on its Q (their slots are freed by the previous item's MMAs),
      // so those go out first and the wait for the Q buffer comes after them. Items without keys take no part
      // in this (no Q tile, zeros stored straight from registers), so the barrier completes exactly once per Q
      // tile and this warp is never more than one phase away from it.
      bool q_pending = false;
      if (item != first_item) {
        cur = describe(item);
        q_pending = cur.list_len > 0;
        if constexpr (!kPacked && !kDense) {
          list_ids = (lane < cur.list_len) ? __ldg(p.col_idx + cur.list_begin + lane) : 0;
        }
      }
      auto settle_q = [&]() -> bool {
        bool got = true;
        if (q_tiles_done > 0) {
          got = mbar_wait(&sm.q_free, (q_tiles_done - 1) & 1, &sm.abort_flag, p.status, 11);
          got = __all_sync(0xffffffffu, got);
        }
        if (got) issue_q_load(cur);
        q_pending = false;
        return got;
      };
      const int n_entries = entries_of(cur);
      const int num_tiles = tiles_of(cur);
      const int q_at = min(2 * num_tiles, kSlots);
      // load i: K (even) or V (odd) of tile i / 2; a slot is reused every kSlots loads
      for (int i = (item == first_item ? loads_issued : 0); ok && i < 2 * num_tiles; ++i) {
        if (q_pending && i == q_at && !settle_q()) {
          ok = false;
          break;
        }
        const int t = i >> 1;
        int kv_row0, kv_row1 = 0, blocks_here = 1;
        if constexpr (!kPacked) {
          if constexpr (!kDense) {
            // block ids are fetched 32 at a time, one per lane, when the walk enters a new chunk
            const int e = t / kTilesPerBlock;
            if ((i & 1) == 0 && e > 0 && (e & 31) == 0 && t % kTilesPerBlock == 0)
              list_ids = (e + lane < n_entries) ? __ldg(p.col_idx + cur.list_begin + e + lane) : 0;
          }
          kv_row0 = unpacked_row(t);
        } else {
          const int e = kBlocksPerTile * t;
          kv_row0 = static_cast<int>(sm.union_ids[e]) * kBlock;
          if (kBlocksPerTile > 1 && e + 1 < n_entries) {
            // two 32-key blocks side by side in one 64-key tile; an odd union leaves the last tile half filled
            kv_row1 = static_cast<int>(sm.union_ids[e + 1]) * kBlock;
            blocks_here = 2;
          }
        }
        const int g = load0 + i;
        const int slot = g % kSlots;
        TL(20 + (i & 1));
        if (g >= kSlots) {
          ok = mbar_wait(&sm.done[slot], ((g / kSlots) - 1) & 1, &sm.abort_flag, p.status, 10);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        issue_load(cur, slot, i & 1, kv_row0, kv_row1, blocks_here);
        TL(22);
      }
      if (ok && q_pending) ok = settle_q();
      if constexpr (!kMultiItem) break;
      load0 += 2 * num_tiles;
      if (num_tiles > 0) ++q_tiles_done;
    }
  } else if (warp == 5) {
    // =============================== UMMA issuer ========================================
    // descriptor low words: Q is fixed; K/V slots differ only in their base address
    const uint32_t q_lo0 = umma_desc_lo(smem_u32(sm.q[0]), 16);
    const uint32_t kv_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), 16);            // as K (K-major)
    const uint32_t v_lo0 = umma_desc_lo(smem_u32(sm.kv[0][0]), kTileN * 128);   // as V (MN-major)
    constexpr uint32_t slot_step = (2 * kTileN * 64 * 2) >> 4;                  // 16 KB per ring slot
    TL_DECL(1)
    bool ok = true;
    int load0 = 0, tile0 = 0, q_loads = 0;   // loads / tiles / Q tiles of earlier items
    for (int item = first_item; ok && item < n_items; item += gridDim.x) {
      if (item != first_item) cur = describe(item);
      const int num_tiles = tiles_of(cur);
      if (num_tiles == 0) {
        if constexpr (!kMultiItem) break;
        continue;
      }
      // S_t = Q K_t^T into S buffer (tile0 + t) & 1
      auto issue_qk = [&](int t) -> bool {
        const int g = load0 + 2 * t;
        const int slot = g % kSlots;
        TL(10);
        bool got = mbar_wait(&sm.kv_full[slot], (g / kSlots) & 1, &sm.abort_flag, p.status, 21);
        got = __all_sync(0xffffffffu, got);
        if (!got) return false;
        TL(11);
        issue_qk64(tmem + kColS + ((tile0 + t) & 1) * kTileN, q_lo0, kv_lo0 + slot * slot_step, &sm.done[slot]);
        TL(12);
        return true;
      };
      ok = mbar_wait(&sm.q_full, q_loads & 1, &sm.abort_flag, p.status, 20);
      ok = __all_sync(0xffffffffu, ok);
      ++q_loads;
      ok = ok && issue_qk(0);
      for (int t = 0; ok && t < num_tiles; ++t) {
        // The S buffer of tile t+1 last held P of the tile two before it, whose P V was issued
        // earlier by this thread, and tcgen05 operations of one thread execute in issue order.
        if (t + 1 < num_tiles && !issue_qk(t + 1)) {
          ok = false;
          break;
        }
        const int g = load0 + 2 * t + 1;
        const int slot = g % kSlots;
        const int gt = tile0 + t;
        TL(13);
        ok = mbar_wait2(&sm.p_full[gt & 1], (gt >> 1) & 1, &sm.kv_full[slot], (g / kSlots) & 1, &sm.abort_flag,
                        p.status, 22);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        TL(14);
        // the first P V of an item overwrites O: the softmax warps handed P over after they had read the
        // previous item's O out in their epilogue
        issue_pv64(tO, tmem + kColS + (gt & 1) * kTileN, v_lo0 + slot * slot_step, t > 0, &sm.done[slot]);
        TL(15);
      }
      if constexpr (!kMultiItem) break;
      load0 += 2 * num_tiles;
      tile0 += num_tiles;
    }
  } else {
    // =============================== softmax / epilogue =================================
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const float scale_log2 = p.scale_log2;
    // packed walk: this warp's 32 rows belong to one query block
    const int my_group = kPacked ? (warp * 32) / kBlock : 0;
    bool ok = true;
    TL_DECL(0)
    int load0 = 0, tile0 = 0;   // loads / tiles of earlier items
    [[maybe_unused]] Item nxt = cur;   // multi-item: the next item's row_ptr entries are fetched one item ahead
    for (int item = first_item; ok && item < n_items; item += gridDim.x) {
      if constexpr (kMultiItem) {
        cur = nxt;
        if (item + static_cast<int>(gridDim.x) < n_items) nxt = describe(item + gridDim.x);
      }
      const int n_entries = entries_of(cur);
      const int num_tiles = tiles_of(cur);
      const bool group_valid = my_group < cur.groups_here;
      RowState st{-INFINITY, 0.f};
      // One 64-key tile of the softmax.
      auto tile_body = [&](int t) -> bool {
        TL(1);
        // S_t is ready when the Q K^T batch that read ring load 2t of this item has completed
        const int gk = load0 + 2 * t;
        if (!mbar_wait(&sm.done[gk % kSlots], (gk / kSlots) & 1, &sm.abort_flag, p.status, 30)) return false;
        TL(2);
        tc_fence_after();
        const int buf = (tile0 + t) & 1;   // S buffer of the tile
        const uint32_t tS = tmem + kColS + buf * kTileN + lane_base;
        // packed walk: which 32-column chunks of this tile hold key blocks this warp's query block kept
        bool keep0 = true, keep1 = true;
        if constexpr (kPacked) {
          const int e = kBlocksPerTile * t;
          const int id0 = sm.union_ids[e];
          keep0 = group_valid && ((sm.member[my_group][id0 >> 5] >> (id0 & 31)) & 1u) != 0u;
          if constexpr (kBlocksPerTile == 1) {
            keep1 = keep0;
          } else {
            keep1 = false;
            if (e + 1 < n_entries) {
              const int id1 = sm.union_ids[e + 1];
              keep1 = group_valid && ((sm.member[my_group][id1 >> 5] >> (id1 & 31)) & 1u) != 0u;
            }
          }
        }
        uint32_t pk[32];
        if (kPacked && !keep0 && !keep1) {
          // nothing of this tile is kept by this warp's query block: P = 0, no exponentials
#pragma unroll
          for (int j = 0; j < 32; ++j) pk[j] = 0u;
        } else {
          uint32_t r0[32], r1[32];
          tmem_ld32(tS, r0);
          tmem_ld32(tS + 32, r1);
          tmem_wait_ld();
          TL(3);
          if constexpr (kDense) {
            const int valid_cols = p.seq_len - t * kTileN;   // ragged tail of the sequence
            if (valid_cols < kTileN) mask_columns_from(r0, r1, valid_cols);
          }
          if constexpr (kPacked) {
            if (!keep0) {
#pragma unroll
              for (int j = 0; j < 32; ++j) r0[j] = 0xff800000u;   // -inf
            }
            if (!keep1) {
#pragma unroll
              for (int j = 0; j < 32; ++j) r1[j] = 0xff800000u;
            }
          }
          float2 sums;
          bool exact = (st.m == -INFINITY);   // nothing accumulated yet: no reference maximum to try
          if (!__all_sync(0xffffffffu, exact)) {
            sums = softmax_group_fast(r0, r1, scale_log2, st.m, pk);
            exact = !(sums.x + sums.y <= 256.0f);   // logits outgrew the running maximum (or NaN)
          }
          if (__any_sync(0xffffffffu, exact)) {
            const float alpha = softmax_group_exact(r0, r1, scale_log2, st, pk, sums);
            if (t > 0) {
              // O must be quiescent: wait until P_{t-1} V_{t-1} (which read ring load 2t-1) has drained
              const int gp = load0 + 2 * (t - 1) + 1;
              if (!mbar_wait(&sm.done[gp % kSlots], (gp / kSlots) & 1, &sm.abort_flag, p.status, 32)) return false;
              tc_fence_after();
              rescale_accumulator_row(tO + lane_base, alpha);
              if (p.slow_path_events != nullptr && lane == 0) atomicAdd(p.slow_path_events, 1ull);
            }
          }
          st.l += sums.x + sums.y;
        }
        TL(4);
        tmem_st32(tS, pk);  // P_t over the first 32 columns of S_t
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_full[buf]);
        TL(5);
        return true;
      };
      for (int t = 0; ok && t < num_tiles; ++t) ok = tile_body(t);
      if constexpr (kDense) {
        // ---- epilogue of the dense walk: O / l -> bf16 -> global, each row from its own thread ----------
        // (with the staged epilogue of the other walks its main loop compiled 1-2 % slower, measured, and its
        // epilogue is 0.3 % of a 64k launch)
        if (!ok) break;
        if (num_tiles > 0) {
          const int gl = load0 + 2 * (num_tiles - 1) + 1;   // the last P V read this load's slot
          ok = mbar_wait(&sm.done[gl % kSlots], (gl / kSlots) & 1, &sm.abort_flag, p.status, 31);
        }
        tc_fence_after();
        const int row = cur.q_row0 + tid;
        const bool row_valid = row < p.seq_len;
        const float inv_l = st.l > 0.f ? (1.f / st.l) : 0.f;
        __nv_bfloat16* o_row = reinterpret_cast<__nv_bfloat16*>(p.o) + cur.batch * p.o_stride_b +
                               cur.head * p.o_stride_h + static_cast<int64_t>(row) * p.o_stride_t;
        store_output_row(tO + lane_base, num_tiles > 0, inv_l, o_row, row_valid);
        if (p.lse != nullptr && row_valid)
          p.lse[static_cast<int64_t>(cur.bh) * p.seq_len + row] = (st.m + log2f(st.l)) * 0.69314718055994531f;
      } else {
        // ---- epilogue: O / l -> bf16 -> shared memory -> global (an empty list gives zeros) ----------
        // Every thread goes through the barrier below even after a wait has run out (it then stages zeros), so
        // that none is left waiting there; what is done after it is decided by the shared flag.
        if (ok && num_tiles > 0) {
          const int gl = load0 + 2 * (num_tiles - 1) + 1;   // the last P V read this load's slot
          ok = mbar_wait(&sm.done[gl % kSlots], (gl / kSlots) & 1, &sm.abort_flag, p.status, 31);
        }
        tc_fence_after();
        const float inv_l = st.l > 0.f ? (1.f / st.l) : 0.f;
        if (num_tiles == 0) {
          // no keys: zeros, straight from registers (the Q buffer may already hold a later item's tile)
          const int row = cur.q_row0 + tid;
          __nv_bfloat16* o_row = reinterpret_cast<__nv_bfloat16*>(p.o) + cur.batch * p.o_stride_b +
                                 cur.head * p.o_stride_h + static_cast<int64_t>(row) * p.o_stride_t;
          store_output_row(0u, false, 0.f, o_row, row < p.seq_len);
        } else {
          // The Q tile is dead (the item's last Q K^T completed before its last P V did): it stages the output.
          stage_output_row(tO + lane_base, ok, inv_l, &sm.q[0][0], tid);
          named_barrier_sync(1, kSoftmaxThreads);
          if (*reinterpret_cast<volatile int*>(&sm.abort_flag) != 0) break;
          if (tid == 0) {
            // rows beyond the sequence end are clipped by the tensor map
            tma_store_4d(&tm_o, sm.q[0], 0, cur.q_row0, cur.head, cur.batch);
            tma_store_4d(&tm_o, sm.q[1], 64, cur.q_row0, cur.head, cur.batch);
            tma_store_commit();
            tma_store_wait_read();
            if constexpr (kMultiItem) mbar_arrive(&sm.q_free);
          }
        }
      }
      if constexpr (!kMultiItem) break;
      tc_fence_before();   // the next item's first P V overwrites O: order these reads before its hand-over
      load0 += 2 * num_tiles;
      tile0 += num_tiles;
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

template <int kBlock, bool kDense, bool kMultiItem>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                   const AttnParams& p, int batch, cudaStream_t stream) {
  auto kernel = attn_kernel<kBlock, kDense, kMultiItem>;
  const int smem = static_cast<int>(sizeof(AttnSmem<kBlock>));
  static SmemLimit limit;  // per template instantiation
  cudaError_t e = ensure_dynamic_smem(kernel, smem, limit);
  if (e != cudaSuccess) return e;
  // one CTA per item, or (kMultiItem and p.max_ctas > 0) at most that many CTAs, each running through its
  // share of the items
  long long ctas = p.num_items;
  if (ctas <= 0) return cudaSuccess;
  if (kMultiItem && p.max_ctas > 0 && ctas > p.max_ctas) ctas = p.max_ctas;
  kernel<<<static_cast<unsigned>(ctas), kThreads, smem, stream>>>(tq, tk, tv, to, p);
  return cudaGetLastError();
}

}  // namespace

int attn_sparse_max_blocks(int block_size) { return block_size < kTileM ? kMaxPackedBlocks : 16384; }

// Tensor maps: Q and O boxes 64 x 128 rows, K and V boxes 64 x min(64, block_size) rows.
// p.num_q_tiles = ceil(seq_len / 128), p.num_blocks = seq_len / block_size.
cudaError_t launch_attn_sparse(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const CUtensorMap& to, const AttnParams& p, int batch, int block_size,
                               cudaStream_t stream) {
  if (block_size == 128) return launch<128, false, true>(tq, tk, tv, to, p, batch, stream);
  if (block_size == 64) return launch<64, false, false>(tq, tk, tv, to, p, batch, stream);
  return launch<32, false, false>(tq, tk, tv, to, p, batch, stream);
}

// Tensor maps: Q and O boxes 64 x 128 rows, K and V boxes 64 x 64 rows. p.num_q_tiles = ceil(seq_len / 128).
cudaError_t launch_attn_dense(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                              const CUtensorMap& to, const AttnParams& p, int batch, cudaStream_t stream) {
  return launch<128, true, false>(tq, tk, tv, to, p, batch, stream);
}

}  // namespace sparsed
