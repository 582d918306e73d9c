// Device-side building blocks shared by the attention kernels (dense and block-sparse):
// the single-pass online softmax of one query row over a 64-key group of logits held in
// registers, the rescaling of the output accumulator in tensor memory, the recording of the
// per-group row statistics the switch step pools into A', and the output epilogue.
//
// The softmax works on base-2 logits against a STALE running maximum: a group is exponentiated
// once, p = 2^(s * scale - m), without first taking the group's maximum. A row sum <= 2^8 proves
// that no p exceeded 2^8, so m is still a safe reference (bf16 P and the fp32 accumulators have
// ample headroom); otherwise (first group, or logits that outgrew m) the caller takes the exact
// path: true maximum of the group, the group redone against it, and everything accumulated so
// far rescaled by 2^(m_old - m_new).
#pragma once

#include "sm100_primitives.cuh"

namespace sparsed {

// Running softmax state of one query row.
struct RowState {
  float m;  // reference maximum in use (base-2 logits), -inf before the first group
  float l;  // sum of p accumulated so far, relative to m
};

// -inf in the columns at and beyond `valid_cols` of a 64-column group (ragged tails, masked blocks).
__device__ __forceinline__ void mask_columns_from(uint32_t (&r0)[32], uint32_t (&r1)[32], int valid_cols) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    if (j >= valid_cols) r0[j] = 0xff800000u;
    if (32 + j >= valid_cols) r1[j] = 0xff800000u;
  }
}

// Fast path. r0 / r1: logits of columns 0-31 / 32-63. Writes P as bf16 pairs (pk[j] = columns
// 2j, 2j+1) and returns the sums of p over columns 0-31 and 32-63. Every exponential is one
// ex2.approx (moving a quarter or a half of them to an FMA-pipe polynomial was measured and lost
// 4 % and 10 %: the softmax warps are bound by instruction issue and latency, not by the SFU).
__device__ __forceinline__ float2 softmax_group_fast(const uint32_t (&r0)[32], const uint32_t (&r1)[32],
                                                     float scale_log2, float m, uint32_t (&pk)[32]) {
  const float2 sc = make_float2(scale_log2, scale_log2);
  const float2 nm = make_float2(-m, -m);
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
  return make_float2(acc0.x + acc0.y, acc1.x + acc1.y);
}

// Exact path: adopts the group's true maximum where it exceeds st.m, redoes the group against
// the (possibly new) st.m and returns the factor by which everything accumulated before this
// group (st.l, already scaled here, and the caller's output accumulator) has to be multiplied.
// An all -inf group of a row that has seen nothing yet keeps m = -inf and gives p = 0.
__device__ __forceinline__ float softmax_group_exact(const uint32_t (&r0)[32], const uint32_t (&r1)[32],
                                                     float scale_log2, RowState& st, uint32_t (&pk)[32],
                                                     float2& sums) {
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j) mx = fmaxf(mx, fmaxf(__uint_as_float(r0[j]), __uint_as_float(r1[j])));
  const float m_group = mx * scale_log2;
  float alpha = 1.f;
  if (m_group > st.m) {
    alpha = fast_exp2(st.m - m_group);  // 0 when nothing was accumulated yet
    st.m = m_group;
    st.l *= alpha;
  }
  // a row whose logits so far are all -inf: use 0 as the reference so that 2^(-inf - 0) = 0, not NaN
  const float m_ref = st.m == -INFINITY ? 0.f : st.m;
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float p0 = fast_exp2(fmaf(__uint_as_float(r0[2 * j]), scale_log2, -m_ref));
    const float p1 = fast_exp2(fmaf(__uint_as_float(r0[2 * j + 1]), scale_log2, -m_ref));
    s0 += p0;
    s0 += p1;
    pk[j] = pack_bf16x2(p0, p1);
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float p0 = fast_exp2(fmaf(__uint_as_float(r1[2 * j]), scale_log2, -m_ref));
    const float p1 = fast_exp2(fmaf(__uint_as_float(r1[2 * j + 1]), scale_log2, -m_ref));
    s1 += p0;
    s1 += p1;
    pk[16 + j] = pack_bf16x2(p0, p1);
  }
  sums = make_float2(s0, s1);
  return alpha;
}

// Multiplies this thread's row of a 128-column fp32 accumulator in tensor memory by alpha.
// The accumulator must be quiescent (every MMA that writes it has completed).
__device__ __forceinline__ void rescale_accumulator_row(uint32_t t_acc_row, float alpha) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t o[32];
    tmem_ld32(t_acc_row + c * 32, o);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
    tmem_st32(t_acc_row + c * 32, o);
  }
}

// Row statistics for the switch step: log2 of the sum of 2^(scaled logit) of one query row over
// each group of `stat_keys` keys (32, 64 or 128), laid out [batch*head][128-row query tile]
// [key group][row in tile] so that a query tile's statistics are one contiguous run. The
// attention kernels feed it 64 keys at a time (the two 32-column sums of a softmax group,
// relative to the reference maximum in use at that moment).
template <int kStatKeys>   // 0 = no statistics, else 32, 64 or 128 keys per statistic
struct RowStatWriter {
  float* next;       // where this row's next statistic goes (statistics of one row are 128 floats apart)
  int left;          // statistics still to be written for this row (0 for rows beyond the sequence end)
  float carry;       // 128-key groups: sum of the group's first 64-key half, relative to the CURRENT reference maximum
  float lg0, lg1;    // log2 of the sums of the group in flight (begin -> finish)

  // first: the row's first statistic, or null for a row beyond the sequence end; n_groups = ceil(seq_len / kStatKeys)
  __device__ __forceinline__ void init(float* first, int n_groups) {
    next = first;
    left = first != nullptr ? n_groups : 0;
    carry = 0.f;
    lg0 = lg1 = 0.f;
  }
  // The caller's reference maximum moved (exact path): everything summed so far shrinks by alpha = 2^(m_old - m_new).
  __device__ __forceinline__ void rescale(float alpha) {
    if constexpr (kStatKeys == 128) carry *= alpha;
  }
  // Two halves, because a warp issues in order: `begin` only STARTS the logarithm(s) as soon as the sums
  // exist; `finish`, called after P has been handed over (by then the results are there), adds the
  // reference maximum and stores. Every instruction here is paid by the softmax warps, the busiest
  // warps of the kernel, hence the running pointer and counter instead of index arithmetic, and a carry that
  // is kept relative to the current maximum (rescaled on the rare exact path) instead of being converted
  // with an exponential on every second tile.
  // second_half: 128-key groups only: this is the second 64-key tile of its group; sums: the tile's two
  // 32-column sums relative to the current reference maximum.
  __device__ __forceinline__ void begin(float2 sums, bool second_half) {
    if constexpr (kStatKeys == 64) {
      lg0 = fast_log2(sums.x + sums.y);
    } else if constexpr (kStatKeys == 32) {
      lg0 = fast_log2(sums.x);
      lg1 = fast_log2(sums.y);
    } else if constexpr (kStatKeys == 128) {
      carry += sums.x + sums.y;
      if (second_half) {
        lg0 = fast_log2(carry);
        carry = 0.f;
      }
    }
  }
  // m: the reference maximum the sums given to `begin` were relative to.
  // (a group that lies wholly beyond a ragged sequence end has no statistic: `left` runs out first)
  __device__ __forceinline__ void finish(float m, bool second_half) {
    if constexpr (kStatKeys == 64) {
      if (left > 0) __stcs(next, m + lg0);
      next += 128;
      --left;
    } else if constexpr (kStatKeys == 32) {
      if (left > 0) __stcs(next, m + lg0);
      if (left > 1) __stcs(next + 128, m + lg1);
      next += 256;
      left -= 2;
    } else if constexpr (kStatKeys == 128) {
      if (second_half) {
        if (left > 0) __stcs(next, m + lg0);
        next += 128;
        --left;
      }
    }
  }
};

// O / l -> bf16, this thread's row, straight from tensor memory to global memory.
// t_acc_row: the row's tensor-memory address; have_acc = false writes zeros (empty key list).
__device__ __forceinline__ void store_output_row(uint32_t t_acc_row, bool have_acc, float inv_l, __nv_bfloat16* o_row,
                                                 bool row_valid) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t r[32];
    if (have_acc) {
      tmem_ld32(t_acc_row + c * 32, r);
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
}

// O / l -> bf16, this thread's row, from tensor memory into a shared-memory tile from which a TMA store
// writes the whole 128-row tile out. (Storing each row from its own thread instead - 32 different cache lines
// per warp instruction - was measured at about 6000 clocks per 128-row tile.)
// tile: 128 rows x 128 columns of bf16 as two 64-column halves of 128 rows x 128 bytes (16 KB each, 1024-byte
// aligned), 128-byte swizzle as the tensor maps use it: the 16-byte chunk c of row r sits at chunk c ^ (r & 7).
// t_acc_row: the row's tensor-memory address; have_acc = false writes zeros (empty key list).
__device__ __forceinline__ void stage_output_row(uint32_t t_acc_row, bool have_acc, float inv_l, __nv_bfloat16* tile,
                                                 int row) {
  uint8_t* base = reinterpret_cast<uint8_t*>(tile) + row * 128;
  const int sw = row & 7;
#pragma unroll
  for (int c = 0; c < 4; ++c) {   // 32 columns each: chunks 4 (c & 1) .. +3 of half c >> 1
    uint32_t r[32];
    if (have_acc) {
      tmem_ld32(t_acc_row + c * 32, r);
      tmem_wait_ld();
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) r[j] = 0u;
    }
    uint8_t* half = base + (c >> 1) * (128 * 128);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint4 out;
      out.x = pack_bf16x2(__uint_as_float(r[8 * g + 0]) * inv_l, __uint_as_float(r[8 * g + 1]) * inv_l);
      out.y = pack_bf16x2(__uint_as_float(r[8 * g + 2]) * inv_l, __uint_as_float(r[8 * g + 3]) * inv_l);
      out.z = pack_bf16x2(__uint_as_float(r[8 * g + 4]) * inv_l, __uint_as_float(r[8 * g + 5]) * inv_l);
      out.w = pack_bf16x2(__uint_as_float(r[8 * g + 6]) * inv_l, __uint_as_float(r[8 * g + 7]) * inv_l);
      *reinterpret_cast<uint4*>(half + (((4 * (c & 1) + g) ^ sw) << 4)) = out;
    }
  }
  fence_proxy_async_smem();   // the TMA store reads these writes through the async proxy
}

// ------------------------------------------------------------------------------------------
// UMMA issue helpers for 64-key tiles of 128B-swizzled shared memory (head_dim 128 as two 64-wide
// halves). Called by a converged warp; one elected lane issues. `done` receives one arrival when
// these MMAs (and everything the lane issued before them) have completed: the same barrier tells
// the softmax threads that their input is ready and the producer that the operand's ring slot is
// free again, so each batch costs a single tcgen05.commit (an expensive instruction: measured at
// about 150 clocks of the issuing thread).
// ------------------------------------------------------------------------------------------
struct UmmaTile64 {
  static constexpr int kKeys = 64;
  static constexpr uint32_t kHi = umma_desc_hi_sw128(1024);
  static constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 64, false, false);   // S = Q K^T, both K-major
  static constexpr uint32_t kIdescPV = umma_idesc_bf16(128, 128, false, true);   // O += P V, V MN-major
  static constexpr uint32_t kQHalfStep = (128 * 64 * 2) >> 4;                    // 16 KB per head_dim half of Q
  static constexpr uint32_t kHalfStep = (kKeys * 64 * 2) >> 4;                   // 8 KB per head_dim half of a tile
};

// S[tmem_s] = Q K^T: eight M128 N64 K16 MMAs. q_lo / k_lo: low descriptor words of the two operands.
__device__ __forceinline__ void issue_qk64(uint32_t tmem_s, uint32_t q_lo, uint32_t k_lo, uint64_t* done) {
  tc_fence_after();
  if (elect_one_sync()) {
    umma_ss_words<false>(tmem_s, q_lo, UmmaTile64::kHi, k_lo, UmmaTile64::kHi, UmmaTile64::kIdescQK);
#pragma unroll
    for (int kk = 1; kk < 8; ++kk) {
      umma_ss_words<true>(tmem_s, q_lo + (kk >> 2) * UmmaTile64::kQHalfStep + (kk & 3) * 2, UmmaTile64::kHi,
                          k_lo + (kk >> 2) * UmmaTile64::kHalfStep + (kk & 3) * 2, UmmaTile64::kHi,
                          UmmaTile64::kIdescQK);
    }
    umma_commit(done);
  }
  __syncwarp();
}

// O[tmem_o] (+)= P[tmem_p] V: four M128 N128 K16 MMAs with P (bf16 pairs) read from tensor memory.
// v_lo: low descriptor word of the V tile as an MN-major operand (16 keys are 2048 bytes apart).
__device__ __forceinline__ void issue_pv64(uint32_t tmem_o, uint32_t tmem_p, uint32_t v_lo, bool accumulate,
                                           uint64_t* done) {
  tc_fence_after();
  if (elect_one_sync()) {
    umma_ts_words(tmem_o, tmem_p, v_lo, UmmaTile64::kHi, UmmaTile64::kIdescPV, accumulate ? 1u : 0u);
#pragma unroll
    for (int kk = 1; kk < 4; ++kk)
      umma_ts_words(tmem_o, tmem_p + kk * 8, v_lo + kk * 128, UmmaTile64::kHi, UmmaTile64::kIdescPV, 1u);
    umma_commit(done);
  }
  __syncwarp();
}

}  // namespace sparsed
