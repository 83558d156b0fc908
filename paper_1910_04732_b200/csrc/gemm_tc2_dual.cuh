// Two-configuration form of the grouped CTA-pair GEMM (gemm_tc2_group.cuh): one persistent launch whose
// problems are of TWO kinds, each with its own operand majors and epilogue, fixed at compile time.
//
// Why: the backward pass of the gated factorized layer has two steps whose products are independent of
// each other but of different kinds --
//   first  : dH' = dY P       (A K-major, B MN-major, bf16 store)  and  dP = dY^T H'          (both MN-major, weight-gradient epilogue)
//   second : dX = dH' (zQ)    (A K-major, B MN-major, bf16 store)  and  dQ = diag(z) dH'^T X  (both MN-major, weight-gradient epilogue)
// Launched kind by kind, the weight gradients are few long tiles (162 tiles of 64 k-blocks on 74 pairs at
// BERT sizes: 2.2 rounds, the third round a fifth full) next to many short ones.  In one work list the
// longest-first schedule fills every pair evenly, and a launch boundary per step disappears.
//
// The kind is a property of the work item, so every role branches once per ITEM into a loop compiled for
// that kind; the loops themselves are those of gemm2_group_kernel.  (Taking majors or epilogue kind at run
// time inside the loops was measured: the MMA issue loop alone lost 10 % to a single run-time condition.)
#pragma once
#include "gemm_tc2_group.cuh"

namespace flop {
namespace tc {

struct PairBars {
  uint32_t base;
  __device__ __forceinline__ uint32_t full(int s) const { return base + 8u * (uint32_t)s; }
  __device__ __forceinline__ uint32_t empty(int s) const { return base + 8u * (uint32_t)(kMaxStages + s); }
  __device__ __forceinline__ uint32_t tfull(int a) const { return base + 8u * (uint32_t)(2 * kMaxStages + a); }
  __device__ __forceinline__ uint32_t tempty(int a) const { return base + 8u * (uint32_t)(2 * kMaxStages + 2 + a); }
  __device__ __forceinline__ uint32_t exit_bar() const { return base + 8u * (uint32_t)(2 * kMaxStages + 4); }
};

// TMA producer: the k-blocks of one work item (both CTAs of the pair run this for their halves).
template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool pair_produce_item(const GroupParams& gp, const GroupItem& it, uint32_t rank, uint32_t smem_base,
                                                  uint32_t sbytes, const PairBars& bars, int& stage, uint32_t& phase,
                                                  volatile int* abort_flag) {
  const GroupProblem& pr = gp.prob[it.g];
  const int half_n = pr.p.bn >> 1;
  const uint32_t tx = kATileBytes + (uint32_t)half_n * BK * 2;
  const int m_base = it.tm * BM2 + (int)rank * BM;
  const int n_base = it.tn * pr.p.bn + (int)rank * half_n;
  for (int kb = it.kb0; kb < it.kb1; ++kb) {
    if (!mbar_wait2(bars.empty(stage), phase ^ 1u, abort_flag)) return false;
    const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
    const uint32_t fb = map_to_cta(bars.full(stage), 0);    // the leader's barrier
    mbar_expect_tx_cluster(fb, tx);
    if (!A_MN) {
      tma_load_2d_pair(sa, &pr.ta, kb * BK, m_base, fb);
    } else {
#pragma unroll
      for (int i = 0; i < BM / (int)kBoxMN; ++i)
        tma_load_2d_pair(sa + i * kBoxBytes, &pr.ta, m_base + i * (int)kBoxMN, kb * BK, fb);
    }
    if (!B_MN) {
      tma_load_2d_pair(sb, &pr.tb, kb * BK, n_base, fb);
    } else {
      for (int i = 0; i < half_n / (int)kBoxMN; ++i)
        tma_load_2d_pair(sb + i * kBoxBytes, &pr.tb, n_base + i * (int)kBoxMN, kb * BK, fb);
    }
    if (++stage == gp.stages) { stage = 0; phase ^= 1u; }
  }
  return true;
}

// MMA issuer (leader CTA, one thread): the k-blocks of one work item into accumulator buffer `acc`.
template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool pair_mma_item(const GroupParams& gp, const GroupItem& it, uint32_t smem_base, uint32_t sbytes,
                                              const PairBars& bars, uint32_t tmem_base, int& stage, uint32_t& phase, int& acc,
                                              uint32_t& acc_phase, volatile int* abort_flag) {
  const uint32_t idesc = instr_desc2(A_MN, B_MN, gp.prob[it.g].p.bn);
  if (!mbar_wait2(bars.tempty(acc), acc_phase ^ 1u, abort_flag)) return false;
  tcgen05_fence_after();
  const uint32_t d_tmem = tmem_base + (uint32_t)acc * acc_stride(gp.bn_max);
  for (int kb = it.kb0; kb < it.kb1; ++kb) {
    if (!mbar_wait2(bars.full(stage), phase, abort_flag)) return false;
    tcgen05_fence_after();
    const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
#pragma unroll
    for (int k = 0; k < BK / UMMA_K; ++k) {
      const uint64_t ad = smem_desc(sa + (A_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), A_MN);
      const uint64_t bd = smem_desc(sb + (B_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), B_MN);
      umma2_bf16(d_tmem, ad, bd, idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
    }
    umma2_commit_mc(bars.empty(stage), 3);    // frees the stage in both CTAs
    if (++stage == gp.stages) { stage = 0; phase ^= 1u; }
  }
  umma2_commit_mc(bars.tfull(acc), 3);        // accumulator halves complete in both CTAs
  if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
  return true;
}

// Kind 0 problems use <A0, B0, E0>, kind 1 problems <A1, B1, E1> (Params::kind).
template <bool A0, bool B0, int E0, bool A1, bool B1, int E1>
__global__ void __launch_bounds__(kThreads, 1)
gemm2_dual_kernel(const __grid_constant__ GroupParams gp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sbytes = stage_bytes2(gp.bn_max);
  const uint32_t store_base = smem_base + (uint32_t)gp.stages * sbytes;
  const PairBars bars{store_base + kStoreBufTotal};
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WorkRange wr = work_range(gp, pair, npairs);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < gp.stages; ++s) { mbar_init(bars.full(s), 2); mbar_init(bars.empty(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bars.tfull(a), 1); mbar_init(bars.tempty(a), 2 * kEpiWarps); }
    mbar_init(bars.exit_bar(), 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane < gp.n) {
    prefetch_tmap(&gp.prob[lane].ta);
    prefetch_tmap(&gp.prob[lane].tb);
    if (gp.prob[lane].p.tma_store) prefetch_tmap(&gp.prob[lane].tout);
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
  if (gp.stamp && blockIdx.x == 0 && threadIdx.x == 0) gp.stamp[0] = global_ns();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
        const GroupItem it = work_item(gp, wi, BM2);
        if (!it.active) continue;
        if (gp.prob[it.g].p.kind == 0) ok = pair_produce_item<A0, B0>(gp, it, rank, smem_base, sbytes, bars, stage, phase, abort_flag);
        else                           ok = pair_produce_item<A1, B1>(gp, it, rank, smem_base, sbytes, bars, stage, phase, abort_flag);
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
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
        const GroupItem it = work_item(gp, wi, BM2);
        if (!it.active) continue;
        if (gp.prob[it.g].p.kind == 0)
          ok = pair_mma_item<A0, B0>(gp, it, smem_base, sbytes, bars, tmem_base, stage, phase, acc, acc_phase, abort_flag);
        else
          ok = pair_mma_item<A1, B1>(gp, it, smem_base, sbytes, bars, tmem_base, stage, phase, acc, acc_phase, abort_flag);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps (both CTAs)
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
      const GroupItem it = work_item(gp, wi, BM2);
      if (!it.active) continue;
      const Params& p = gp.prob[it.g].p;
      if (!mbar_wait2(bars.tfull(acc), acc_phase, abort_flag)) { ok = false; }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t sbuf = store_base + (uint32_t)(warp - 2) * kStoreBufBytes, t_acc = tmem_base + (uint32_t)acc * acc_stride(gp.bn_max);
      const int row0 = it.tm * BM2 + (int)rank * BM;
      const uint32_t rel = map_to_cta(bars.tempty(acc), 0);
      if (p.kind == 0) run_epilogue<E0, true>(p, &gp.prob[it.g].tout, sbuf, t_acc, row0, it.tn * p.bn, it.n_limit, it.split, it.tn, warp, lane, rel);
      else             run_epilogue<E1, true>(p, &gp.prob[it.g].tout, sbuf, t_acc, row0, it.tn * p.bn, it.n_limit, it.split, it.tn, warp, lane, rel);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();
  }
  // ---------------------------------------------------------------- teardown (as in gemm2_group_kernel)
  tcgen05_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_arrive_cluster(map_to_cta(bars.exit_bar(), 0));
    mbar_arrive_cluster(map_to_cta(bars.exit_bar(), 1));
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster_acq(bars.exit_bar(), 0)) {
      if (clock64() - t0 > kWaitCycles) { report_timeout(); break; }
    }
  }
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc2(tmem_base, kTmemCols);
  }
  if (gp.stamp && threadIdx.x == 0) atomicMax(gp.stamp + 1, global_ns());
}

}  // namespace tc
}  // namespace flop
