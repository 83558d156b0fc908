// Chained form of the two-configuration CTA-pair GEMM (gemm_tc2_dual.cuh): ONE persistent launch for GEMM
// stages that feed each other.
//
// The gated factorized layer (Section 4.1 of the paper) is two products in the forward pass,
//     H' = (X Q^T) * z   ->   Y = H' P^T,
// and four in the backward pass, two of which read the output of another,
//     dH' = dY P  (and dP = dY^T H')   ->   dX = dH' (diag(z) Q)  and  dQ = diag(z) dH'^T X.
// Launched stage by stage, every boundary costs a pipeline drain, a launch gap and a pipeline fill on all
// 148 SMs, and the small kernels around the products (diag(z) Q, the second stage of dlog_alpha) sit on the
// critical path.  Here the tiles of both stages are in one work list.  A tile that reads another problem's
// output waits for it through counters in global memory:
//   * every epilogue warp of a producing tile, once its part of the tile is written (bulk stores complete),
//     adds one to sig[tm] of its problem, tm = the 256-row block of the tile;
//   * the TMA producer of a consuming tile waits (bounded) until the counter of the row block it is about
//     to read has reached 16 x the number of N tiles of the producing problem: before the first k-block
//     when the A operand is a row block of the producer's output (Y = H' P^T, dX), before every fourth
//     k-block when the contraction runs over the producer's rows (dQ contracts over tokens);
//   * only the TMA producer waits -- MMA issuer and epilogue warps follow through the pipeline barriers, so
//     the issue loop is untouched.
// The pairs draw their tiles from one queue in which every first-stage tile comes before every second-stage
// tile (the host orders it), first-stage tiles wait for nothing, and all CTAs of the launch are resident at
// once (one per SM): a drawn tile only waits for tiles that are already being worked on, so every wait ends.
// All the same every wait is bounded and records FLOP_ERR_TIMEOUT.
//
// Folded into the launch as well:
//   * diag(z) Q (the B operand of dX) is formed by two helper warps per CTA while the first-stage tiles run,
//     and guarded by one more counter (the epilogue warps cannot do it on the side: the work is a chain of
//     dependent memory round trips, and the first accumulators would wait for them);
//   * the second stage of dlog_alpha: the partial row dots <Q[k,:], (dH'^T X)[k,:]> of a 32-row slab are
//     added, in fixed order, by whichever epilogue warp finishes the slab's last N tile (a counter per
//     slab), so the result does not depend on which warp that is.
// The counters live in a caller-provided, zero-initialised sync area; the last unit to finish clears it
// again, so that the next launch (or the next replay of a captured graph) finds it zeroed.
#pragma once
#include "gemm_tc2_dual.cuh"

namespace flop {
namespace tc {

// words of the sync area with a fixed meaning; the per-problem counters follow
constexpr int kSyncDone = 0;     // units that have finished (the last one clears the area)
constexpr int kSyncAbort = 1;    // set when a wait of this launch gave up: the other units stop waiting
constexpr int kSyncSide = 2;     // helper warps that have finished their share of diag(z) Q
constexpr int kSyncWork = 3;     // tickets handed out by the launch's work queue
constexpr int kSyncFixed = 4;
constexpr int kQueueSlots = 8;   // depth of the per-pair ring through which the leader hands queue entries to the other roles
constexpr unsigned kSigPerTile = 2 * kEpiWarps;   // arrivals per 256-row tile: both CTAs' epilogue warps

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned atom_acq_rel_add(unsigned* p, unsigned v) {
  unsigned old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
// orders accesses through the asynchronous proxy (TMA) against those through the generic proxy
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait until *ctr >= need.  Returns false if it gave up, or if another unit of the launch did.
// No proxy fence on this side: what the waiting thread goes on to read, it reads with TMA loads, and the data
// was either written by TMA stores whose completion the writer awaited, or by ordinary stores that the
// writer fenced towards the asynchronous proxy, before the writer's release.  (A proxy fence here would also
// drain the TMA loads this thread has in flight, once per work item.)
__device__ __forceinline__ bool chain_wait(const unsigned* ctr, unsigned need, unsigned* sync, volatile int* abort_flag) {
  if (ld_acquire_u32(ctr) >= need) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (ld_acquire_u32(ctr) >= need) return true;
    __nanosleep(64);
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (ld_acquire_u32(sync + kSyncAbort) != 0u) { *abort_flag = 1; return false; }
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        atomicExch(sync + kSyncAbort, 1u);
        report_timeout();
        return false;
      }
    }
  }
}

// N tiles of problem-size N that exist this launch (a device-side size may shorten it; 0 counts as 1).
__device__ __forceinline__ unsigned active_tiles_n(int n_cap, int bn, const int* dyn_n) {
  const int n_eff = dyn_n ? max(1, min(n_cap, __ldg(dyn_n))) : n_cap;
  return (unsigned)((n_eff + bn - 1) / bn);
}

struct ChainProducerState { bool side_ok; };

// TMA producer of one work item, with the waits on other problems' outputs (both CTAs of the pair run this).
template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool chain_produce_item(const GroupParams& gp, const GroupItem& it, uint32_t rank, uint32_t smem_base,
                                                   uint32_t sbytes, const PairBars& bars, int& stage, uint32_t& phase,
                                                   volatile int* abort_flag, ChainProducerState& cs) {
  const GroupProblem& pr = gp.prob[it.g];
  const ChainLink& ln = pr.p.link;
  const int half_n = pr.p.bn >> 1;
  const uint32_t tx = kATileBytes + (uint32_t)half_n * BK * 2;
  const int m_base = it.tm * BM2 + (int)rank * BM;
  const int n_base = it.tn * pr.p.bn + (int)rank * half_n;
  if (ln.side_dep && !cs.side_ok) {       // the B operand is formed by this launch's side work
    if (!chain_wait(gp.sync + kSyncSide, gp.side_need, gp.sync, abort_flag)) return false;
    cs.side_ok = true;
  }
  unsigned need = 0;
  int known_rb = -1;                      // producer row blocks up to here are known to be complete
  if (ln.dep) {
    need = kSigPerTile * active_tiles_n(ln.dep_n_cap, ln.dep_bn, ln.dep_dyn_n);
    if (ln.dep_mode == 1) {
      if (!chain_wait(ln.dep + it.tm, need, gp.sync, abort_flag)) return false;
    }
  }
  for (int kb = it.kb0; kb < it.kb1; ++kb) {
    if (ln.dep && ln.dep_mode == 2) {     // the contraction runs over the producer's rows: 64 per k-block
      const int rb = (kb * BK) / BM2;
      if (rb > known_rb) {
        if (!chain_wait(ln.dep + rb, need, gp.sync, abort_flag)) return false;
        known_rb = rb;
      }
    }
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

// What an epilogue warp does after the tile's epilogue proper: publish the tile to its consumers, and add up
// the dlog_alpha partials of its 32-row slab if it is the last to finish there.
template <int EPI>
__device__ __forceinline__ void chain_after_tile(const Params& p, const GroupItem& it, uint32_t rank, int row0, int warp, int lane) {
  const ChainLink& ln = p.link;
  if (ln.sig) {
    if (p.tma_store) {
      if (lane == 0) { tma_store_wait_all(); fence_proxy_async_all(); }   // the bulk stores have been written, not just read
    } else {
      fence_proxy_async_all();
      __threadfence();
    }
    __syncwarp();
    if (lane == 0) red_release_add(ln.sig + it.tm, 1u);
  }
  if (EPI == EPI_WGRAD && ln.fin && p.qdot) {
    const int q = warp & 3;
    __threadfence();                      // this warp's partial row dots are visible before the arrival
    __syncwarp();
    unsigned* f = ln.fin + ((it.tm * 2 + (int)rank) * 4 + q);
    const unsigned tiles = active_tiles_n(p.N, p.bn, p.dyn_n);
    unsigned old = 0;
    if (lane == 0) old = atom_acq_rel_add(f, 1u);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old + 1u == 2u * tiles) {         // both column halves of every N tile of this slab are in
      __threadfence();
      const int row = row0 + q * 32 + lane;
      if (row < p.M) {
        float s = 0.f;
        for (unsigned pp = 0; pp < 2u * tiles; ++pp) s += __ldcg(p.dz_part + (int64_t)pp * p.dz_stride + row);
        const float v = s * __ldg(ln.dz_dla + row);
        ln.dla[row] = ln.dla_accumulate ? ln.dla[row] + v : v;
      }
    }
  }
}

// diag(z) Q of every problem that asks for it, spread over the helper warps of all CTAs of the launch.  A
// helper thread keeps kSideBatch 16-byte loads in flight (the work is latency-bound: a few units per thread).
constexpr int kSideWarps = 2;
constexpr int kSideBatch = 8;
constexpr int kChainThreads = kThreads + 32 * kSideWarps;

__device__ __forceinline__ void chain_side_work(const GroupParams& gp, int lane) {
  const int64_t first = (int64_t)blockIdx.x * (32 * kSideWarps) + ((int)threadIdx.x - kThreads);
  const int64_t step = (int64_t)gridDim.x * (32 * kSideWarps);
  for (int i = 0; i < gp.n; ++i) {
    const ChainLink& ln = gp.prob[i].p.link;
    if (!ln.sw_qz) continue;
    const int c8 = (ln.sw_cols + 7) >> 3;              // 8 columns (16 bytes) per unit; rows are 16-byte aligned
    const int64_t total = (int64_t)ln.sw_rows * c8;
    for (int64_t u0 = first; u0 < total; u0 += step * kSideBatch) {
      uint4 raw[kSideBatch];
      float g[kSideBatch];
      int row[kSideBatch], c0[kSideBatch];
#pragma unroll
      for (int b = 0; b < kSideBatch; ++b) {
        const int64_t u = u0 + (int64_t)b * step;
        raw[b] = make_uint4(0u, 0u, 0u, 0u);
        g[b] = 0.f;
        row[b] = -1; c0[b] = 0;
        if (u < total) {
          row[b] = (int)(u / c8);
          c0[b] = (int)(u - (int64_t)row[b] * c8) * 8;
          const __nv_bfloat16* q = ln.sw_q + (int64_t)row[b] * ln.sw_ldq + c0[b];
          g[b] = __ldg(ln.sw_z + row[b]);
          if (c0[b] + 8 <= ln.sw_cols) {
            raw[b] = __ldg(reinterpret_cast<const uint4*>(q));
          } else {                                       // ragged last unit of a row: element by element, here
            __nv_bfloat16* o = ln.sw_qz + (int64_t)row[b] * ln.sw_ldqz + c0[b];
            for (int k = 0; k < ln.sw_cols - c0[b]; ++k) o[k] = __float2bfloat16_rn(__bfloat162float(q[k]) * g[b]);
            row[b] = -1;
          }
        }
      }
#pragma unroll
      for (int b = 0; b < kSideBatch; ++b) {
        if (row[b] < 0) continue;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw[b]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 x = __bfloat1622float2(h[e]);
          h[e] = __floats2bfloat162_rn(x.x * g[b], x.y * g[b]);
        }
        *reinterpret_cast<uint4*>(ln.sw_qz + (int64_t)row[b] * ln.sw_ldqz + c0[b]) = raw[b];
      }
    }
  }
  fence_proxy_async_all();   // the rows just written are read by TMA loads of other CTAs
  __threadfence();
  __syncwarp();
  if (lane == 0) red_release_add(gp.sync + kSyncSide, 1u);
}

// ---------------------------------------------------------------- the launch's work queue
// The tiles are not dealt out in advance.  Equal tiles do not take equal time on every SM (the slowest pair of a
// statically dealt launch finished 12 us after the fastest, of 78), so the pairs draw tiles from one queue: entry
// `pair` first, then entry npairs + ticket with tickets from an atomic counter in the sync area.  The host orders
// the queue (sched.item): every tile after the tiles it waits for -- so a drawn tile only ever waits for tiles that
// some pair is already working on -- and long tiles before short ones.
// The leader's TMA thread draws; every other role of the pair (the peer's TMA thread, the MMA thread, all epilogue
// warps) must walk the same sequence, so the leader publishes each entry through a small ring in the shared memory
// of both CTAs: qfull[s] (one per CTA) says slot s holds the next entry, qempty[s] (in the leader) counts the 18
// readers of the pair.  -1 ends the sequence.
struct QueueRing {
  uint32_t base;   // qfull[kQueueSlots], qempty[kQueueSlots] (8 bytes each), then the slots (4 bytes each)
  __device__ __forceinline__ uint32_t full(int s) const { return base + 8u * (uint32_t)s; }
  __device__ __forceinline__ uint32_t empty(int s) const { return base + 8u * (uint32_t)(kQueueSlots + s); }
  __device__ __forceinline__ uint32_t slot(int s) const { return base + 16u * (uint32_t)kQueueSlots + 4u * (uint32_t)s; }
};
constexpr uint32_t kQueueReaders = 2 * kEpiWarps + 2;   // epilogue warps of both CTAs, the MMA thread, the peer's TMA thread

__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster_acq(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cluster_acq(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        report_timeout();
        return false;
      }
    }
  }
}
__device__ __forceinline__ void st_shared_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}

// Leader's TMA thread: draws the next entry and hands it to the pair.  Returns the work-list index, -1 when the
// queue is exhausted, -2 when a wait gave up.  The first two entries of a pair are fixed (queue positions pair and
// npairs + pair); from the third on the position is 2 * npairs + ticket, with `ticket` drawn one call ahead, so
// that the atomic's latency overlaps the loads of a tile.
// Cost: release / acquire operations at cluster scope cost the issuing thread the better part of a microsecond
// each (measured), per tile and per reader.  So the leader's own readers (the MMA thread above all) are served
// with CTA-scope operations on the leader's copy of the ring, and the peer's copy is written with ONE
// asynchronous remote store that also completes the peer's barrier (st.async ... complete_tx): the leader never
// waits for the peer.  The peer's TMA thread arms its barriers (arrive.expect_tx, 4 bytes) one use ahead.  The
// wait for a free slot needs no acquire: the readers publish nothing with their arrivals.
__device__ __forceinline__ int queue_draw(const GroupParams& gp, const QueueRing& q, int& cursor, int pair, int npairs, unsigned& ticket,
                                          volatile int* abort_flag) {
  const int s = cursor & (kQueueSlots - 1);
  const uint32_t use = (uint32_t)(cursor / kQueueSlots) & 1u;
  if (!mbar_wait(q.empty(s), use ^ 1u, abort_flag)) return -2;     // the readers of the slot's previous entry are done
  const int pos = cursor == 0 ? pair : cursor == 1 ? npairs + pair : 2 * npairs + (int)ticket;
  const int idx = pos < gp.total_work ? work_at(gp, pos) : -1;
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(q.slot(s)), "r"((uint32_t)idx) : "memory");
  mbar_arrive(q.full(s));                                          // release at CTA scope: the leader's readers
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];"
               ::"r"(map_to_cta(q.slot(s), 1)), "r"((uint32_t)idx), "r"(map_to_cta(q.full(s), 1)) : "memory");
  if (idx >= 0 && cursor >= 1) ticket = atomicAdd(gp.sync + kSyncWork, 1u);   // for the draw after the next
  ++cursor;
  return idx;
}
// Every other role (one thread per reader): the next entry of the pair's sequence.  `rearm`: the peer's TMA
// thread arms the slot's barrier for its next use before it hands the slot back.
__device__ __forceinline__ int queue_next(const QueueRing& q, int& cursor, uint32_t rank, bool rearm, volatile int* abort_flag) {
  const int s = cursor & (kQueueSlots - 1);
  const uint32_t use = (uint32_t)(cursor / kQueueSlots) & 1u;
  if (!mbar_wait(q.full(s), use, abort_flag)) return -2;
  const int idx = (int)ld_shared_u32(q.slot(s));
  if (rank == 0) {
    mbar_arrive(q.empty(s));
  } else {
    if (rearm) mbar_expect_tx(q.full(s), 4u);
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(map_to_cta(q.empty(s), 0)) : "memory");
  }
  ++cursor;
  return idx;
}

// Kind 0 problems use <A0, B0, E0>, kind 1 problems <A1, B1, E1> (Params::kind).
template <bool A0, bool B0, int E0, bool A1, bool B1, int E1>
__global__ void __launch_bounds__(kChainThreads, 1)
gemm2_chain_kernel(const __grid_constant__ GroupParams gp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sbytes = stage_bytes2(gp.bn_max);
  const uint32_t store_base = smem_base + (uint32_t)gp.stages * sbytes;
  const PairBars bars{store_base + kStoreBufTotal};
  const QueueRing queue{bars.exit_bar() + 8u};
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ int s_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    s_abort = 0;
    s_last = 0;
    for (int s = 0; s < gp.stages; ++s) { mbar_init(bars.full(s), 2); mbar_init(bars.empty(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bars.tfull(a), 1); mbar_init(bars.tempty(a), 2 * kEpiWarps); }
    mbar_init(bars.exit_bar(), 2);
    for (int s = 0; s < kQueueSlots; ++s) { mbar_init(queue.full(s), 1); mbar_init(queue.empty(s), kQueueReaders); }
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
      ChainProducerState cs{false};
      int cursor = 0;
      unsigned ticket = 0;
      // The leader keeps the ring one entry ahead of its own loads: the entry of the next tile is published before
      // the loads of the current one, so that no reader (the peer's TMA thread least of all) learns of a tile late.
      if (rank != 0)
        for (int s = 0; s < kQueueSlots; ++s) mbar_expect_tx(queue.full(s), 4u);     // first use of every slot
      int w = rank == 0 ? queue_draw(gp, queue, cursor, pair, npairs, ticket, abort_flag) : queue_next(queue, cursor, rank, true, abort_flag);
      while (ok && w >= 0) {
        int w_next = -1;
        if (rank == 0) w_next = queue_draw(gp, queue, cursor, pair, npairs, ticket, abort_flag);
        const GroupItem it = decode_group(gp, w, BM2);
        if (it.active) {
          if (gp.prob[it.g].p.kind == 0) ok = chain_produce_item<A0, B0>(gp, it, rank, smem_base, sbytes, bars, stage, phase, abort_flag, cs);
          else                           ok = chain_produce_item<A1, B1>(gp, it, rank, smem_base, sbytes, bars, stage, phase, abort_flag, cs);
        }
        if (rank != 0 && ok) w_next = queue_next(queue, cursor, rank, true, abort_flag);
        w = w_next;
      }
      if (w == -2) ok = false;
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
      int cursor = 0;
      while (ok) {
        const int w = queue_next(queue, cursor, 0u, false, abort_flag);
        if (w < 0) break;
        const GroupItem it = decode_group(gp, w, BM2);
        if (!it.active) continue;
        if (gp.prob[it.g].p.kind == 0)
          ok = pair_mma_item<A0, B0>(gp, it, smem_base, sbytes, bars, tmem_base, stage, phase, acc, acc_phase, abort_flag);
        else
          ok = pair_mma_item<A1, B1>(gp, it, smem_base, sbytes, bars, tmem_base, stage, phase, acc, acc_phase, abort_flag);
      }
    }
  } else if (warp >= 2 + kEpiWarps) {
    // ------------------------------------------------------------ helper warps (both CTAs): side work, then done
    if (gp.side_need) chain_side_work(gp, lane);
  } else {
    // ------------------------------------------------------------ epilogue warps (both CTAs)
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    int cursor = 0;
    while (ok) {
      int w = 0;
      if (lane == 0) w = queue_next(queue, cursor, rank, false, abort_flag);    // one lane reads the ring: the warp cannot disagree
      w = __shfl_sync(0xffffffffu, w, 0);
      if (w < 0) break;
      const GroupItem it = decode_group(gp, w, BM2);
      if (!it.active) continue;
      const Params& p = gp.prob[it.g].p;
      if (!mbar_wait2(bars.tfull(acc), acc_phase, abort_flag)) { ok = false; }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t sbuf = store_base + (uint32_t)(warp - 2) * kStoreBufBytes, t_acc = tmem_base + (uint32_t)acc * acc_stride(gp.bn_max);
      const int row0 = it.tm * BM2 + (int)rank * BM;
      const uint32_t rel = map_to_cta(bars.tempty(acc), 0);
      if (p.kind == 0) {
        run_epilogue<E0, true>(p, &gp.prob[it.g].tout, sbuf, t_acc, row0, it.tn * p.bn, it.n_limit, it.split, it.tn, warp, lane, rel);
        chain_after_tile<E0>(p, it, rank, row0, warp, lane);
      } else {
        run_epilogue<E1, true>(p, &gp.prob[it.g].tout, sbuf, t_acc, row0, it.tn * p.bn, it.n_limit, it.split, it.tn, warp, lane, rel);
        chain_after_tile<E1>(p, it, rank, row0, warp, lane);
      }
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
    // Both CTAs of this pair are past their last wait and their last arrival on the launch's counters.  The
    // unit that arrives last knows that every unit is: it clears the sync area for the next launch.
    if (rank == 0) {
      __threadfence();
      if (atom_acq_rel_add(gp.sync + kSyncDone, 1u) + 1u == (unsigned)npairs) s_last = 1;
    }
  }
  __syncthreads();
  if (s_last) {
    for (int i = threadIdx.x; i < gp.sync_words; i += blockDim.x) gp.sync[i] = 0u;
  }
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc2(tmem_base, kTmemCols);
  }
  if (gp.stamp && threadIdx.x == 0) atomicMax(gp.stamp + 1, global_ns());
}

}  // namespace tc
}  // namespace flop
