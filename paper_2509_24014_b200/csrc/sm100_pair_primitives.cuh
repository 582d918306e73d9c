// Inline-PTX wrappers for kernels whose tensor-core instructions span a PAIR of CTAs on neighbouring
// SMs (tcgen05 with cta_group::2, launched as clusters of two): cluster rank and barrier, addresses
// and arrivals in the peer CTA's shared memory, TMA loads that signal a barrier of the peer CTA,
// tensor-memory allocation for the pair, and UMMA issue / commit for M = 256 tiles.
//
// Device status code 4 (beside the codes of sm100_primitives.cuh) = the two CTAs of a pair got different
// tensor-memory bases and did no work.
//
// A kernel uses either these or the cta_group::1 wrappers of sm100_primitives.cuh for its tcgen05
// allocation, MMA and commit instructions, never both. Every CTA loads its own tiles: no load here delivers to more than one CTA.
#pragma once

#include "sm100_primitives.cuh"

namespace sparsed {

__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// Cluster-wide barrier in two halves; every thread of both CTAs executes both, in converged code.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// The shared::cluster address of this CTA's shared-memory address `smem_addr` in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}

__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t cluster_addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}

// One arrival on an mbarrier given by its shared::cluster address (this CTA's or the peer's). Default
// semantics (release at CTA scope): a cluster-scope release makes the arriving thread wait for all of its earlier
// global stores, which the callers here neither need nor can afford; what they hand over lives in tensor memory
// and is ordered by the tcgen05 fences around the arrival.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// 4-D tiled TMA load into THIS CTA's shared memory whose completion bytes are counted on a barrier
// that may live in the peer CTA (given as a shared::cluster address); the data go to this CTA alone.
// Coordinates are innermost first; c0 * sizeof(element) must be a multiple of 16.
__device__ __forceinline__ void tma_load_4d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, "
      "%5, %6}], [%2];"
      :
      : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(c0), "r"(c1),
        "r"(c2), "r"(c3)
      : "memory");
}

// Tensor memory for the pair: the same warp of BOTH CTAs executes each of these; both get the same base.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem] over the CTA pair (M = 256: each CTA supplies its 128 rows of A and half of
// B's N rows from the same shared-memory offsets, and holds its 128 rows of D). Issued by one thread of the
// leader CTA. Descriptors as (lo, hi) words.
template <bool kAccumulate>
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                             uint32_t b_hi, uint32_t idesc) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      ".reg .b64 da, db;\n"
      "setp.ne.b32 p, %6, 0;\n"
      "mov.b64 da, {%1, %2};\n"
      "mov.b64 db, {%3, %4};\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n"
      "}\n"
      :
      : "r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(kAccumulate ? 1 : 0)
      : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem] over the CTA pair; each CTA reads A from its own tensor memory.
__device__ __forceinline__ void umma_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      ".reg .b64 db;\n"
      "setp.ne.b32 p, %5, 0;\n"
      "mov.b64 db, {%2, %3};\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n"
      "}\n"
      :
      : "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

// One arrival on the barrier at this shared-memory offset in EACH CTA of the pair once every tcgen05
// operation issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  const uint16_t both = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"(both)
      : "memory");
}

}  // namespace sparsed
