// On-chip forward chain of the gated factorized layer (Section 4.1 of the paper: y = P G Q x is two products; after
// pruning they are "much smaller (but still dense)" products of width k): Y = ((X Q^T) * z) P^T in ONE launch in
// which the rank-k intermediate H' never leaves the SM.
//
// One CTA owns 128 token rows and a slice of the output columns:
//   phase 1  H = X_rows Q^T: X tiles [128 x 64] and Q tiles [k_pad x 64] arrive by TMA in a two-stage ring, one thread
//            issues tcgen05.mma (fp32 accumulators in tensor memory, columns 0..k_pad-1; k_pad <= 512 = all of
//            tensor memory, two instructions per k-step when k_pad > 256)
//   phase 2  the eight epilogue warps read the accumulator (tcgen05.ld), apply the gate, round to bf16 and write H'
//            into shared memory in the 128-byte-swizzled K-major layout the tensor core reads its A operand in
//            (k_pad/64 panels of 128 rows x 128 bytes); the panels take the place of the phase-1 stages
//   phase 3  Y_tile = H' P_tile^T for the CTA's N tiles: P tiles [128 x 64] stream through a ring of their own
//            (two to eight stages, whatever the phase-1 ring leaves; its loads start at kernel entry: nothing
//            aliases them), accumulators alternate between two tensor-memory buffers (free again once phase 2 has
//            read H), the epilogue stages bf16 blocks in shared memory and writes them with TMA stores
// The price is that every CTA of a row block recomputes H (the slices of a row block do not share it), so the chain
// pays when the first product is cheap next to the second or when there are enough row blocks to need few slices;
// the host decides (flop_lib.cu) and the two-launch path stays the default elsewhere.
// Roles, descriptors, epilogue and bounded waits are those of gemm_tc.cuh.
#pragma once
#include "gemm_tc.cuh"

namespace flop {
namespace tc {

constexpr int kChainMaxK = 512;                         // k_pad: columns of tensor memory / 64-column panels of shared memory for H'
constexpr int kChainBN = 128;                           // N tile of the second product
constexpr int kChainStages1 = 2;                        // phase-1 ring: X tile (16 KB) + Q tile (k_pad x 128 B) per stage
constexpr uint32_t kChainStage3Bytes = kChainBN * BK * 2;              // 16 KB
constexpr int kChainMaxStages3 = 8;
constexpr uint32_t kChainRingBytes = 192 * 1024;        // phase-1 ring (later the H' panels) + phase-3 ring
constexpr uint32_t kChainSmemBytes = 1024 + kChainRingBytes + kStoreBufTotal + 256;
__host__ __device__ inline uint32_t chain_stage1_bytes(int k_pad) { return kATileBytes + (uint32_t)k_pad * BK * 2; }
__host__ __device__ inline int chain_stages3(int k_pad) {
  const int n = (int)((kChainRingBytes - kChainStages1 * chain_stage1_bytes(k_pad)) / kChainStage3Bytes);
  return n < kChainMaxStages3 ? n : kChainMaxStages3;    // k_pad = 512: 2 stages; 384: 4; <= 256: 6 and more
}

struct ChainFwdParams {
  CUtensorMap tx, tq, tp, ty;     // X [T, d_in] box 64x128; Q [k, d_in] box 64x64; P [d_out, k] box 64x128; Y [T, d_out] box 64x32
  Params y;                       // epilogue of the second product (bf16 store of Y through the staged TMA path)
  const float* z;                 // gate of H's columns (nullable: compact factors carry it already)
  int T, d_in, d_out, k, k_pad;   // k_pad = k rounded up to 64
  int tiles_n, tiles_per_cta;     // N tiles of Y; consecutive tiles one CTA (blockIdx.x) takes
};

__global__ void __launch_bounds__(kThreads, 1)
chain_fwd_kernel(const __grid_constant__ ChainFwdParams cp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage1_bytes = chain_stage1_bytes(cp.k_pad);
  const int stages3 = chain_stages3(cp.k_pad);
  const uint32_t h_base = smem_base;                                   // phase-1 stages, later the H' panels (k_pad x 256 B <= 2 stages)
  const uint32_t s3_base = smem_base + kChainStages1 * stage1_bytes;
  const uint32_t store_base = smem_base + kChainRingBytes;
  const uint32_t bar_base = store_base + kStoreBufTotal;
  auto full1 = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty1 = [&](int s) { return bar_base + 8u * (uint32_t)(2 + s); };
  auto full3 = [&](int s) { return bar_base + 8u * (uint32_t)(4 + s); };
  auto empty3 = [&](int s) { return bar_base + 8u * (uint32_t)(4 + kChainMaxStages3 + s); };
  auto tfull = [&](int a) { return bar_base + 8u * (uint32_t)(4 + 2 * kChainMaxStages3 + a); };
  auto tempty = [&](int a) { return bar_base + 8u * (uint32_t)(6 + 2 * kChainMaxStages3 + a); };
  const uint32_t h_full = bar_base + 8u * (uint32_t)(8 + 2 * kChainMaxStages3);      // the accumulator of the first product is complete
  const uint32_t h_ready = h_full + 8u;                                              // H' is in shared memory (and tensor memory is free again)
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tm = blockIdx.y;
  const int tn0 = (int)blockIdx.x * cp.tiles_per_cta;
  const int tn1 = min(tn0 + cp.tiles_per_cta, cp.tiles_n);
  const int nkb1 = (cp.d_in + BK - 1) / BK, nkb3 = cp.k_pad / BK;
  const int boxes_q = cp.k_pad / 64;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < kChainStages1; ++s) { mbar_init(full1(s), 1); mbar_init(empty1(s), 1); }
    for (int s = 0; s < stages3; ++s) { mbar_init(full3(s), 1); mbar_init(empty3(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull(a), 1); mbar_init(tempty(a), kEpiWarps); }
    mbar_init(h_full, 1);
    mbar_init(h_ready, kEpiWarps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    prefetch_tmap(&cp.tx); prefetch_tmap(&cp.tq); prefetch_tmap(&cp.tp); prefetch_tmap(&cp.ty);
  }
  if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      // phase 1: X and Q k-blocks
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t tx1 = kATileBytes + (uint32_t)cp.k_pad * BK * 2;
      for (int kb = 0; kb < nkb1 && ok; ++kb) {
        if (!mbar_wait(empty1(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t sa = h_base + (uint32_t)stage * stage1_bytes, sb = sa + kATileBytes;
        mbar_expect_tx(full1(stage), tx1);
        tma_load_2d(sa, &cp.tx, kb * BK, tm * BM, full1(stage));
        for (int i = 0; i < boxes_q; ++i) tma_load_2d(sb + (uint32_t)i * kBoxBytes, &cp.tq, kb * BK, i * 64, full1(stage));
        if (++stage == kChainStages1) { stage = 0; phase ^= 1u; }
      }
      // phase 3: P k-blocks of every N tile of this CTA (their ring aliases nothing, so they run ahead of phase 2)
      stage = 0; phase = 0;
      for (int tn = tn0; tn < tn1 && ok; ++tn) {
        for (int kb = 0; kb < nkb3; ++kb) {
          if (!mbar_wait(empty3(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(full3(stage), kChainStage3Bytes);
          tma_load_2d(s3_base + (uint32_t)stage * kChainStage3Bytes, &cp.tp, kb * BK, tn * kChainBN, full3(stage));
          if (++stage == stages3) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        const long long t0 = clock64();     // leaving early: let the copies already issued land
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      bool ok = true;
      int stage = 0;
      uint32_t phase = 0;
      const int n_lo = min(cp.k_pad, 256), n_hi = cp.k_pad - n_lo;      // columns 0..255 and 256..k_pad-1 of H
      const uint32_t idesc_lo = instr_desc(false, false, n_lo), idesc_hi = n_hi > 0 ? instr_desc(false, false, n_hi) : 0u;
      for (int kb = 0; kb < nkb1 && ok; ++kb) {
        if (!mbar_wait(full1(stage), phase, abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t sa = h_base + (uint32_t)stage * stage1_bytes, sb = sa + kATileBytes;
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          const uint64_t ad = smem_desc(sa + k * (UMMA_K * 2), false);
          umma_bf16(tmem_base, ad, smem_desc(sb + k * (UMMA_K * 2), false), idesc_lo, (kb > 0 || k > 0) ? 1u : 0u);
          if (n_hi > 0)
            umma_bf16(tmem_base + 256u, ad, smem_desc(sb + 256u * 128u + k * (UMMA_K * 2), false), idesc_hi, (kb > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(empty1(stage));
        if (++stage == kChainStages1) { stage = 0; phase ^= 1u; }
      }
      if (ok) {
        umma_commit(h_full);
        // phase 3 starts when H' is in shared memory; by then the accumulator columns have been read, too
        if (!mbar_wait(h_ready, 0u, abort_flag)) ok = false;
        tcgen05_fence_after();
      }
      const uint32_t idesc3 = instr_desc(false, false, kChainBN);
      stage = 0; phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tn = tn0; tn < tn1 && ok; ++tn) {
        if (!mbar_wait(tempty(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kChainBN);
        for (int kb = 0; kb < nkb3; ++kb) {
          if (!mbar_wait(full3(stage), phase, abort_flag)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t sa = h_base + (uint32_t)kb * kATileBytes, sb = s3_base + (uint32_t)stage * kChainStage3Bytes;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(d_tmem, smem_desc(sa + k * (UMMA_K * 2), false), smem_desc(sb + k * (UMMA_K * 2), false), idesc3,
                      (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(empty3(stage));
          if (++stage == stages3) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    bool ok = mbar_wait(h_full, 0u, abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      // phase 2: accumulator -> gate -> bf16 -> H' panels.  Warp (q, h): rows q*32 + lane, panels h, h + 2, ...
      tcgen05_fence_after();
      const int q = warp & 3, h = (warp - 2) >> 2;
      const int r = q * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
      for (int j = h; j < nkb3; j += 2) {
        uint32_t v0[32], v1[32];
        tmem_ld32(t_row + (uint32_t)(j * 64), v0);
        tmem_ld32(t_row + (uint32_t)(j * 64 + 32), v1);
        tmem_ld_wait();
        const uint32_t row_addr = h_base + (uint32_t)j * kATileBytes + (uint32_t)r * 128u;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint32_t (&v)[32] = half ? v1 : v0;
          const int c0 = j * 64 + half * 32;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int c = c0 + 8 * i + 2 * e;
              float a = __uint_as_float(v[8 * i + 2 * e]), b = __uint_as_float(v[8 * i + 2 * e + 1]);
              if (cp.z) {
                a *= c < cp.k ? __ldg(cp.z + c) : 0.f;
                b *= c + 1 < cp.k ? __ldg(cp.z + c + 1) : 0.f;
              }
              __nv_bfloat162 hh = __floats2bfloat162_rn(a, b);
              pk[e] = *reinterpret_cast<uint32_t*>(&hh);
            }
            st_shared_v4(row_addr + (uint32_t)(((half * 4 + i) ^ (lane & 7)) << 4), pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      fence_async_smem();            // the panels are read by the tensor core (asynchronous proxy)
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(h_ready);
      // phase 3 epilogues
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tn = tn0; tn < tn1 && ok; ++tn) {
        if (!mbar_wait(tfull(acc), acc_phase, abort_flag)) { ok = false; }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tcgen05_fence_after();
        run_epilogue<EPI_STORE, false>(cp.y, &cp.ty, store_base + (uint32_t)(warp - 2) * kStoreBufBytes,
                                       tmem_base + (uint32_t)(acc * kChainBN), tm * BM, tn * kChainBN, cp.d_out, 0, tn, warp, lane, tempty(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    if (lane == 0) tma_store_wait_all();
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace flop
