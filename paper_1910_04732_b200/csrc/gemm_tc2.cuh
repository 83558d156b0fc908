// Two-CTA variant of the bf16 tensor-core GEMM: a cluster of two CTAs (the two SMs of a
// TPC) computes one 256 x BN tile with tcgen05.mma.cta_group::2.
//
// Why: in the one-CTA kernel every SM has to pull a full B tile (BN x 64) per k-block next
// to its A tile, and the measured fill rate of an SM's shared memory (~54 B/clk) is what
// bounds the main loop, not the tensor pipe.  Here each CTA loads its own 128 rows of A but
// only HALF of the B tile (BN/2 rows); the paired MMA reads the two halves from both SMs.
// Bytes per SM per k-block drop from 16 KB + BN*128 to 16 KB + BN*64.
//
// Protocol (rank = position in the pair, rank 0 leads):
//   full[s]    lives in rank 0, expects two arrivals (one arrive.expect_tx per producer) plus
//              the bytes of both CTAs' TMA loads (each load names rank 0's barrier)
//   empty[s]   one per CTA; rank 0's MMA thread releases a stage in both CTAs with one
//              tcgen05.commit ... multicast::cluster
//   tfull[a]   one per CTA, signalled the same way when an accumulator is complete
//   tempty[a]  lives in rank 0, expects the epilogue warps of both CTAs (remote arrivals)
// The accumulator rows 0..127 sit in rank 0's tensor memory, rows 128..255 in rank 1's; each
// CTA's epilogue warps drain their own half.  No TMA load uses multicast.
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
__host__ __device__ inline uint32_t stage_bytes2(int bn) { return kATileBytes + (uint32_t)(bn / 2) * BK * 2; }

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm2_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Params p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sbytes = stage_bytes2(p.bn);
  const uint32_t bar_base = smem_base + (uint32_t)p.stages * sbytes;
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + 2 + a); };
  const uint32_t exit_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages + 4);
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total = p.tiles_m * p.tiles_n * p.splits;
  const int half_n = p.bn >> 1;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * kEpiWarps); }
    mbar_init(exit_bar, 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tmap_a);
    prefetch_tmap(&tmap_b);
  }
  if (warp == 1) tmem_alloc2(smem_u32(&s_tmem_base), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();            // both CTAs' barriers exist before either signals the other
  tcgen05_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = pair; w < total && ok; w += npairs) {
        const WorkItem it = decode(p, w);
        const int m_base = it.tm * BM2 + (int)rank * BM;
        const int n_base = it.tn * p.bn + (int)rank * half_n;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait2(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
          const uint32_t fb = map_to_cta(full_bar(stage), 0);    // the leader's barrier
          mbar_expect_tx_cluster(fb, sbytes);
          if (!A_MN) {
            tma_load_2d_pair(sa, &tmap_a, kb * BK, m_base, fb);
          } else {
#pragma unroll
            for (int i = 0; i < BM / (int)kBoxMN; ++i)
              tma_load_2d_pair(sa + i * kBoxBytes, &tmap_a, m_base + i * (int)kBoxMN, kb * BK, fb);
          }
          if (!B_MN) {
            tma_load_2d_pair(sb, &tmap_b, kb * BK, n_base, fb);
          } else {
            for (int i = 0; i < half_n / (int)kBoxMN; ++i)
              tma_load_2d_pair(sb + i * kBoxBytes, &tmap_b, n_base + i * (int)kBoxMN, kb * BK, fb);
          }
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        // Leaving early: give the copies already issued time to land (they complete within
        // microseconds) so that nothing writes this CTA's shared memory after it has exited.
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = instr_desc2(A_MN, B_MN, p.bn);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int w = pair; w < total && ok; w += npairs) {
        const WorkItem it = decode(p, w);
        if (!mbar_wait2(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.bn);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait2(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = smem_desc(sa + (A_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), A_MN);
            const uint64_t bd = smem_desc(sb + (B_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), B_MN);
            umma2_bf16(d_tmem, ad, bd, idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
          }
          umma2_commit_mc(empty_bar(stage), 3);    // frees the stage in both CTAs
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma2_commit_mc(tfull_bar(acc), 3);        // accumulator halves complete in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (both CTAs)
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int w = pair; w < total && ok; w += npairs) {
      const WorkItem it = decode(p, w);
      if (!mbar_wait2(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      run_epilogue<EPI, true>(p, tmem_base + (uint32_t)(acc * p.bn), it.tm * BM2 + (int)rank * BM, it.tn * p.bn, it.split, it.tn,
                              warp, lane, map_to_cta(tempty_bar(acc), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  // ---------------------------------------------------------------- teardown
  tcgen05_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    // tell both CTAs that this one is past its last use of the pair's barriers and tensor memory
    mbar_arrive_cluster(map_to_cta(exit_bar, 0));
    mbar_arrive_cluster(map_to_cta(exit_bar, 1));
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster_acq(exit_bar, 0)) {
      if (clock64() - t0 > kWaitCycles) { report_timeout(); break; }
    }
  }
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc2(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace flop
