// Grouped form of the one-CTA tensor-core GEMM: up to kMaxGroup (16) independent problems
// D_g = A_g B_g^T (same operand majors and epilogue kind, any sizes) in ONE persistent launch.
//
// Why: the GEMMs of a BERT- or Transformer-XL-sized factorized matrix are 3-20 GFLOP each,
// about one 128 x 192 tile per SM.  Launched one by one, every kernel pays its own pipeline
// fill (first TMA round trip), epilogue drain and launch gap, and the tensor pipe is busy for
// ~20 % of the kernel.  With the tiles of several independent matrices in one work list, every
// CTA walks several tiles back to back: the producer warp is already fetching the next tile's
// k-blocks (possibly of another matrix) while the MMA warp finishes the current one and the
// epilogue warps drain the previous accumulator, so fill and drain are paid once per launch.
//
// Each problem keeps its own tensor maps, sizes, N tile, split-K factor and epilogue pointers in
// a __grid_constant__ table; shared-memory stages and accumulator buffers are sized for the
// largest N tile of the group.  Roles, barriers, epilogues and bounded waits are described in
// gemm_tc.cuh.  A single GEMM runs as a group of one.
#pragma once
#include "gemm_tc.cuh"
#include "schedule.cuh"

namespace flop {
namespace tc {

constexpr int kMaxGroup = 24;   // the four products of six matrices; 24 x 704 B of kernel parameters (the limit is 32 KB)

struct alignas(64) GroupProblem {
  CUtensorMap ta, tb;
  CUtensorMap tout;   // bf16 output, 64 x 32 boxes (used when p.tma_store)
  Params p;
  int work_begin;   // index of this problem's first work item in the group's list
};

struct GroupParams {
  GroupProblem prob[kMaxGroup];
  int n;            // problems in use
  int total_work;   // sum over problems of tiles_m * tiles_n * splits
  int stages;
  int bn_max;       // largest N tile: sizes the stages and the accumulator buffers
  // Optional device-side stamp of this launch (nullable): [0] = %globaltimer when CTA 0 passes the
  // dependency wait, [1] = the latest %globaltimer at which a CTA finished (atomic max).  Lets a
  // caller time launches that run inside a replayed CUDA graph, where host events cannot be placed.
  unsigned long long* stamp;
  // Chained launches only (gemm_tc2_chain.cuh): the zero-initialised sync area, the words in use (the last
  // unit to finish clears them) and the arrivals that complete the launch's side work (0: none).
  unsigned* sync; int sync_words; unsigned side_need;
  // Which work items each persistent unit walks (schedule.cuh); n_units == 0: round-robin.
  Schedule sched;
};

// The work items of persistent unit `unit` of `nunits`: for (i = first; i < last; i += step) item = work_at(gp, i).
struct WorkRange { int first, last, step; };
__device__ __forceinline__ WorkRange work_range(const GroupParams& gp, int unit, int nunits) {
  if (gp.sched.n_units) return WorkRange{(int)gp.sched.begin[unit], (int)gp.sched.begin[unit + 1], 1};
  return WorkRange{unit, gp.total_work, nunits};
}
__device__ __forceinline__ int work_at(const GroupParams& gp, int i) { return gp.sched.n_units ? (int)gp.sched.item[i] : i; }   // chained launches: plain indices

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct GroupItem { int g, tm, tn, split, kb0, kb1, n_limit; bool active; };

// Work item w of the group; bm = rows of D per tile (128, or 256 for a CTA pair).  When a problem
// carries device-side sizes the item may lie outside the effective extent (active = false: every
// role skips it, so stage and accumulator phases stay in step) or have a shorter K loop.
__device__ __forceinline__ GroupItem decode_problem_item(const GroupParams& gp, int g, int w, int bm) {
  const Params& p = gp.prob[g].p;
  const WorkItem it = decode(p, w - gp.prob[g].work_begin);
  GroupItem o{g, it.tm, it.tn, it.split, it.kb0, it.kb1, p.N, true};
  if (p.dyn_m || p.dyn_n || p.dyn_k) {
    const int m_eff = p.dyn_m ? max(1, min(p.M, __ldg(p.dyn_m))) : p.M;
    const int n_eff = p.dyn_n ? max(1, min(p.N, __ldg(p.dyn_n))) : p.N;
    const int k_eff = p.dyn_k ? max(1, min(p.K, __ldg(p.dyn_k))) : p.K;
    if (p.dyn_n) o.n_limit = min(p.N, (n_eff + 63) & ~63);
    o.kb1 = min(o.kb1, (k_eff + BK - 1) / BK);
    o.active = o.tm * bm < m_eff && o.tn * p.bn < n_eff && o.kb0 < o.kb1;
  }
  return o;
}
__device__ __forceinline__ GroupItem decode_group(const GroupParams& gp, int w, int bm) {
  int g = 0;
  for (int i = 1; i < gp.n && w >= gp.prob[i].work_begin; ++i) g = i;   // work_begin ascends; a group of one needs no step
  return decode_problem_item(gp, g, w, bm);
}
// Entry i of a unit's list.  A schedule table built by the grouped launches carries the problem index in the upper
// five bits of its 16-bit entries (kSchedProblemShift), which saves the walk over the problem table once per tile and
// role; without a table the entry is the work-list index itself.
__device__ __forceinline__ GroupItem work_item(const GroupParams& gp, int i, int bm) {
  if (gp.sched.n_units) {
    const int e = (int)gp.sched.item[i];
    return decode_problem_item(gp, e >> kSchedProblemShift, e & ((1 << kSchedProblemShift) - 1), bm);
  }
  return decode_group(gp, i, bm);
}

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_group_kernel(const __grid_constant__ GroupParams gp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sbytes = stage_bytes(gp.bn_max);
  const uint32_t store_base = smem_base + (uint32_t)gp.stages * sbytes;   // 1024-byte aligned: stages are multiples of 1 KB
  const uint32_t bar_base = store_base + kStoreBufTotal;
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + 2 + a); };
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkRange wr = work_range(gp, (int)blockIdx.x, (int)gridDim.x);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < gp.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), kEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane < gp.n) {
    prefetch_tmap(&gp.prob[lane].ta);
    prefetch_tmap(&gp.prob[lane].tb);
    if (gp.prob[lane].p.tma_store) prefetch_tmap(&gp.prob[lane].tout);
  }
  if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;
  pdl_wait();
  pdl_launch_dependents();
  if (gp.stamp && blockIdx.x == 0 && threadIdx.x == 0) gp.stamp[0] = global_ns();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int armed = 0;
      bool ok = true;
      for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
        const GroupItem it = work_item(gp, wi, BM);
        if (!it.active) continue;
        const GroupProblem& pr = gp.prob[it.g];
        const int bn = pr.p.bn;
        const uint32_t tx = kATileBytes + (uint32_t)bn * BK * 2;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, tx);
          if (!A_MN) {
            tma_load_2d(sa, &pr.ta, kb * BK, it.tm * BM, fb);
          } else {
#pragma unroll
            for (int i = 0; i < BM / (int)kBoxMN; ++i)
              tma_load_2d(sa + i * kBoxBytes, &pr.ta, it.tm * BM + i * (int)kBoxMN, kb * BK, fb);
          }
          if (!B_MN) {
            tma_load_2d(sb, &pr.tb, kb * BK, it.tn * bn, fb);
          } else {
            for (int i = 0; i < bn / (int)kBoxMN; ++i)
              tma_load_2d(sb + i * kBoxBytes, &pr.tb, it.tn * bn + i * (int)kBoxMN, kb * BK, fb);
          }
          if (armed < gp.stages) ++armed;
          if (++stage == gp.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        // Leaving early: wait (bounded) until the copies already issued have landed.
        int s = stage;
        uint32_t ph = phase;
        for (int i = 0; i < armed; ++i) {
          if (--s < 0) { s = gp.stages - 1; ph ^= 1u; }
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(s), ph) && clock64() - t0 < kWaitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
        const GroupItem it = work_item(gp, wi, BM);
        if (!it.active) continue;
        const uint32_t idesc = instr_desc(A_MN, B_MN, gp.prob[it.g].p.bn);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * acc_stride(gp.bn_max);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t sa = smem_base + (uint32_t)stage * sbytes, sb = sa + kATileBytes;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t ad = smem_desc(sa + (A_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), A_MN);
            const uint64_t bd = smem_desc(sb + (B_MN ? k * (UMMA_K * 128) : k * (UMMA_K * 2)), B_MN);
            umma_bf16(d_tmem, ad, bd, idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));
          if (++stage == gp.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int wi = wr.first; wi < wr.last && ok; wi += wr.step) {
      const GroupItem it = work_item(gp, wi, BM);
        if (!it.active) continue;
      const Params& p = gp.prob[it.g].p;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      run_epilogue<EPI, false>(p, &gp.prob[it.g].tout, store_base + (uint32_t)(warp - 2) * kStoreBufBytes, tmem_base + (uint32_t)acc * acc_stride(gp.bn_max), it.tm * BM, it.tn * p.bn, it.n_limit, it.split, it.tn, warp, lane,
                               tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();   // this warp's output blocks are written before the CTA retires
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (gp.stamp && threadIdx.x == 0) atomicMax(gp.stamp + 1, global_ns());
}

}  // namespace tc
}  // namespace flop
