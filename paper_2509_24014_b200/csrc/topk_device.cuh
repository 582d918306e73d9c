// Warp-level isolated top-k of one row of pooled block scores (Eq. 5 / Eq. 6) with the row held
// in shared memory as order-preserving 32-bit keys. Used by the stand-alone selection kernel
// and by the tail of the pooled-scoring kernel.
//
// For each key region (prefill blocks [0,pb), generation blocks [pb,nb)) the k-th largest key
// is found by radix selection, 8 bits per pass over a 256-bin warp histogram in shared
// memory, starting below the bits all keys of the region have in common. The search stops as
// soon as the surviving bucket is exactly as large as the number still to take, and once the
// bucket fits in a warp (<= 32 keys) it is finished by ranking those keys against each other.
// Blocks above the threshold are kept, blocks equal to it lowest index first (ties -> lower
// block index). Kept ids are written in ascending order through ballot prefix sums.
#pragma once

#include <stdint.h>

namespace sparsed {

// Order-preserving map float -> uint32 (larger float -> larger key). NaN ranks lowest,
// -0 equals +0.
__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;  // NaN
  if (u == 0x80000000u) u = 0u;                    // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct RegionThreshold {
  uint32_t prefix;   // threshold key bits under `mask`
  uint32_t mask;     // bits that were decided
  int take_equal;    // how many keys equal to the threshold (under mask) are kept, lowest index first
};

// One warp; keys[0..nb) in shared memory; hist = 256 ints of shared memory owned by this warp.
__device__ __forceinline__ RegionThreshold warp_region_threshold(const uint32_t* keys, int lo, int hi, int kk,
                                                                 int* hist, int lane) {
  RegionThreshold r;
  r.prefix = 0u;
  r.mask = 0u;
  r.take_equal = kk;
  if (kk >= hi - lo) return r;  // everything is kept: mask 0 makes every key "equal", take all
  // bits shared by all keys of the region need no pass
  uint32_t all_and = 0xffffffffu, all_or = 0u;
  for (int i = lo + lane; i < hi; i += 32) {
    const uint32_t k = keys[i];
    all_and &= k;
    all_or |= k;
  }
  all_and = __reduce_and_sync(0xffffffffu, all_and);
  all_or = __reduce_or_sync(0xffffffffu, all_or);
  const uint32_t diff = all_and ^ all_or;
  if (diff == 0u) {  // all keys equal
    r.prefix = all_and;
    r.mask = 0xffffffffu;
    return r;
  }
  int top = 32 - __clz(diff);          // number of low bits that vary
  r.mask = top >= 32 ? 0u : ~((1u << top) - 1u);
  r.prefix = all_and & r.mask;
  int need = kk;
  while (top > 0) {
    const int shift = top > 8 ? top - 8 : 0;
    const int bits = top - shift;
    const uint32_t digit_mask = (1u << bits) - 1u;
#pragma unroll
    for (int b = 0; b < 8; ++b) hist[lane * 8 + b] = 0;
    __syncwarp();
    for (int i = lo + lane; i < hi; i += 32) {
      const uint32_t k = keys[i];
      if ((k & r.mask) == r.prefix) atomicAdd(&hist[(k >> shift) & digit_mask], 1);
    }
    __syncwarp();
    // lane l owns bins 8l .. 8l+7; scan from the top bin down
    int local[8];
    int s = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      local[b] = hist[lane * 8 + b];
      s += local[b];
    }
    int above = s;  // inclusive suffix sum over lanes >= lane
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, above, off);
      if (lane + off < 32) above += v;
    }
    above -= s;  // keys in bins of higher lanes
    // the crossing lane: above < need <= above + s
    const bool mine = (above < need) && (need <= above + s);
    int digit = 0, cnt_above = 0, bucket = 0;
    if (mine) {
      int run = above;
#pragma unroll
      for (int b = 7; b >= 0; --b) {
        if (run < need && need <= run + local[b]) {
          digit = lane * 8 + b;
          cnt_above = run;
          bucket = local[b];
        }
        run += local[b];
      }
    }
    const uint32_t who = __ballot_sync(0xffffffffu, mine);
    const int src = __ffs(who) - 1;
    digit = __shfl_sync(0xffffffffu, digit, src);
    cnt_above = __shfl_sync(0xffffffffu, cnt_above, src);
    bucket = __shfl_sync(0xffffffffu, bucket, src);
    need -= cnt_above;
    r.prefix |= static_cast<uint32_t>(digit) << shift;
    r.mask |= digit_mask << shift;
    top = shift;
    if (bucket == need) break;  // the whole surviving bucket is kept: lower bits do not matter
    __syncwarp();
    if (bucket <= 32 && top > 0) {
      // Finish inside the warp: pull the bucket's keys into lanes (in index order) and rank them.
      uint32_t* cand = reinterpret_cast<uint32_t*>(hist);
      const uint32_t lt_mask = (1u << lane) - 1u;
      int filled = 0;
      for (int base = lo; base < hi; base += 32) {
        const int i = base + lane;
        uint32_t k = 0u;
        bool in_bucket = false;
        if (i < hi) {
          k = keys[i];
          in_bucket = (k & r.mask) == r.prefix;
        }
        const uint32_t b = __ballot_sync(0xffffffffu, in_bucket);
        if (in_bucket) cand[filled + __popc(b & lt_mask)] = k;
        filled += __popc(b);
      }
      __syncwarp();
      const bool have = lane < bucket;
      const uint32_t mine_key = have ? cand[lane] : 0u;
      int rank = 0;  // keys ahead of mine in (key descending, position ascending) order
      for (int j = 0; j < bucket; ++j) {
        const uint32_t kj = __shfl_sync(0xffffffffu, mine_key, j);
        rank += (kj > mine_key) || (kj == mine_key && j < lane);
      }
      const uint32_t pick = __ballot_sync(0xffffffffu, have && rank == need - 1);
      const uint32_t thr = __shfl_sync(0xffffffffu, mine_key, __ffs(pick) - 1);
      const int greater = __popc(__ballot_sync(0xffffffffu, have && mine_key > thr));
      r.prefix = thr;
      r.mask = 0xffffffffu;
      need -= greater;
      __syncwarp();
      break;
    }
  }
  r.take_equal = need;
  return r;
}

// Selects and writes one row. keys: nb keys in shared memory (already written and visible to
// the warp). dst: k_pre + k_gen ids, ascending.
__device__ __forceinline__ void warp_select_row(const uint32_t* keys, int nb, int pb, int k_pre, int k_gen,
                                                int* hist, int32_t* dst, int lane) {
  RegionThreshold th[2];
  th[0] = warp_region_threshold(keys, 0, pb, k_pre, hist, lane);
  __syncwarp();
  th[1] = warp_region_threshold(keys, pb, nb, k_gen, hist, lane);
  const uint32_t lt_mask = (1u << lane) - 1u;
  int run = 0;
  int eq_seen0 = 0, eq_seen1 = 0;
  for (int base = 0; base < nb; base += 32) {
    const int i = base + lane;
    const bool second = i >= pb;  // which region this lane's block is in
    const uint32_t mask = second ? th[1].mask : th[0].mask;
    const uint32_t prefix = second ? th[1].prefix : th[0].prefix;
    bool keep = false, eq = false;
    if (i < nb) {
      const uint32_t km = keys[i] & mask;
      eq = km == prefix;
      keep = km > prefix;
    }
    const uint32_t b_eq = __ballot_sync(0xffffffffu, eq);
    if (b_eq != 0u) {
      // equal keys are taken lowest index first, counted per region (a 32-wide chunk can
      // straddle the region boundary)
      const uint32_t second_lanes = __ballot_sync(0xffffffffu, second);
      const uint32_t b_eq0 = b_eq & ~second_lanes, b_eq1 = b_eq & second_lanes;
      if (eq) {
        const int rank = second ? eq_seen1 + __popc(b_eq1 & lt_mask) : eq_seen0 + __popc(b_eq0 & lt_mask);
        keep = rank < (second ? th[1].take_equal : th[0].take_equal);
      }
      eq_seen0 += __popc(b_eq0);
      eq_seen1 += __popc(b_eq1);
    }
    const uint32_t b_keep = __ballot_sync(0xffffffffu, keep);
    if (keep) dst[run + __popc(b_keep & lt_mask)] = i;
    run += __popc(b_keep);
  }
}

}  // namespace sparsed
