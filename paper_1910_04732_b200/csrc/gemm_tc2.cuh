// Two-CTA variant of the bf16 tensor-core GEMM, shared pieces (the kernel is gemm2_group_kernel
// in gemm_tc2_group.cuh): a cluster of two CTAs (the two SMs of a TPC) computes one 256 x BN tile
// with tcgen05.mma.cta_group::2.
//
// Why: in the one-CTA kernel every SM has to pull a full B tile (BN x 64) per k-block next
// to its A tile, and the measured fill rate of an SM's shared memory (~54 B/clk) is what
// bounds the main loop, not the tensor pipe.  Here each CTA loads its own 128 rows of A but
// only HALF of the B tile (BN/2 rows); the paired MMA reads the two halves from both SMs.
// Bytes per SM per k-block drop from 16 KB + BN*128 to 16 KB + BN*64.
//
// Protocol (rank = position in the pair, rank 0 leads):
//   full[s]    lives in rank 0, expects two arrivals (one relaxed arrive.expect_tx per producer) plus
//              the bytes of both CTAs' TMA loads (each load names rank 0's barrier)
//   empty[s]   one per CTA; rank 0's MMA thread releases a stage in both CTAs with one
//              tcgen05.commit ... multicast::cluster
//   tfull[a]   one per CTA, signalled the same way when an accumulator is complete
//   tempty[a]  lives in rank 0, expects the epilogue warps of both CTAs (remote arrivals)
// The accumulator rows 0..127 sit in rank 0's tensor memory, rows 128..255 in rank 1's; each
// CTA's epilogue warps drain their own half.  Every CTA fetches its own operand tiles; the commit
// above is the only instruction that signals both CTAs at once.
// All mbarrier waits are bounded as in the one-CTA kernel; before tensor memory is freed the
// two CTAs shake hands through an mbarrier (bounded) so that neither signals a peer that has
// already left.
#pragma once
#include "gemm_tc.cuh"

namespace flop {
namespace tc {

constexpr int BM2 = 256;   // rows of D per pair tile

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
  return out;
}
// Relaxed: the producer publishes no memory of its own with this arrival (the TMA engine's
// complete_tx carries the data), so the per-stage loop is not slowed by a cluster-scope release.
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster_acq(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// The pipeline barriers are waited on with the default (CTA-scope) try_wait even when the arrivals
// come from the peer: the data they guard is consumed by the tensor core / written by TMA, not
// read by the waiting thread.
__device__ __forceinline__ bool mbar_wait2(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait(bar, parity, abort_flag);
}
// TMA load whose completion bytes go to a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// One arrival on the barrier at this offset in every CTA of `mask`, once the MMAs issued so far are done.
__device__ __forceinline__ void umma2_commit_mc(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t instr_desc2(bool a_mn, bool b_mn, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM2 >> 4) << 24);
}

// bytes one CTA of the pair loads per stage: its 128 rows of A and half of the B tile
// (rounded up to 1 KB: every stage must start on a swizzle-atom boundary, and half of a 208-column tile is 13 KB)
__host__ __device__ inline uint32_t stage_bytes2(int bn) { return kATileBytes + (((uint32_t)(bn / 2) * BK * 2 + 1023u) & ~1023u); }

}  // namespace tc
}  // namespace flop
