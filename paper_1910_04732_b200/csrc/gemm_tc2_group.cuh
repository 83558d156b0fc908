// Grouped form of the two-CTA tensor-core GEMM (pieces in gemm_tc2.cuh): the 256 x BN tiles of up to
// kMaxGroup independent problems in one persistent launch of CTA pairs.  It combines the two
// measures that matter at BERT / Transformer-XL sizes: several tiles per CTA, so that pipeline
// fill and epilogue drain overlap the next tile's main loop, and half a B tile per SM, so that the
// bytes an SM has to pull from L2 per MMA drop by about 40 % (that fill rate, ~50 B/clk/SM, is what
// bounds the one-CTA 128 x 192 x 768 tile; the pair's main loop runs at 87-89 % of the tensor pipe and
// hardly responds to the bytes loaded).  Problem table, work list and epilogues are
// those of gemm_group_kernel; pair protocol and bounded waits are described in gemm_tc2.cuh.
#pragma once
#include "gemm_tc2.cuh"
#include "gemm_tc_group.cuh"

namespace flop {
namespace tc {

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm2_group_kernel(const __grid_constant__ GroupParams gp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sbytes = stage_bytes2(gp.bn_max);
  const uint32_t store_base = smem_base + (uint32_t)gp.stages * sbytes;   // 1024-byte aligned: stages are multiples of 1 KB
  const uint32_t bar_base = store_base + kStoreBufTotal;
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
  const WorkRange wr = work_range(gp, pair, npairs);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < gp.stages; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * kEpiWarps); }
    mbar_init(exit_bar, 2);
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
        const GroupProblem& pr = gp.prob[it.g];
        const int half_n = pr.p.bn >> 1;
        const uint32_t tx = kATileBytes + (uint32_t)half_n * BK * 2;
        const int m_base = it.tm * BM2 + (int)rank * BM;
        const int n_base = it.tn * pr.p.bn + (int)rank * half_n;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait2(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
          const uint32_t fb = map_to_cta(full_bar(stage), 0);    // the leader's barrier
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
        const uint32_t idesc = instr_desc2(A_MN, B_MN, gp.prob[it.g].p.bn);
        if (!mbar_wait2(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * acc_stride(gp.bn_max);
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
          if (++stage == gp.stages) { stage = 0; phase ^= 1u; }
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
    for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
      const GroupItem it = work_item(gp, wi, BM2);
        if (!it.active) continue;
      const Params& p = gp.prob[it.g].p;
      if (!mbar_wait2(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      run_epilogue<EPI, true>(p, &gp.prob[it.g].tout, store_base + (uint32_t)(warp - 2) * kStoreBufBytes, tmem_base + (uint32_t)acc * acc_stride(gp.bn_max), it.tm * BM2 + (int)rank * BM, it.tn * p.bn, it.n_limit, it.split, it.tn,
                              warp, lane, map_to_cta(tempty_bar(acc), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();
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
  if (gp.stamp && threadIdx.x == 0) atomicMax(gp.stamp + 1, global_ns());
}

}  // namespace tc
}  // namespace flop
