// bf16 tensor-core GEMM for sm_100a, shared pieces: D[M,N] = sum_k A(m,k) B(n,k), fp32 accumulate.
//
// The kernels built from this header (gemm_group_kernel in gemm_tc_group.cuh, one CTA per
// 128 x BN tile; gemm2_group_kernel in gemm_tc2_group.cuh, a CTA pair per 256 x BN tile; and
// gemm2_dual_kernel in gemm_tc2_dual.cuh, the pair kernel for a launch that holds two kinds of problem)
// serve all six GEMMs of the gated factorized layer W = P diag(z) Q (Section 4.1 of the paper).
// Both are persistent and warp-specialised:
//   warp 0      TMA producer: cp.async.bulk.tensor loads (every CTA fetches its own tiles) into a ring of
//               128-byte-swizzled shared-memory stages, completion on mbarriers
//   warp 1      MMA issuer: one thread issues tcgen05.mma (K = 16 per instruction, bf16 in,
//               fp32 accumulators in tensor memory), tcgen05.commit frees stages
//   warps 2..9  epilogue: tcgen05.ld the accumulator (one output row per thread), apply the
//               gate, and either stage bf16 tiles in shared memory for a TMA store, or write
//               weight gradients / fp32 split-K slices directly, with the fused per-row dot
//               product that becomes dz (hence dlog_alpha)
// Two accumulator buffers in tensor memory let the epilogue of one tile overlap the main loop
// of the next.  Operands may be K-major (rows of the row-major matrix run along K) or MN-major
// (the backward GEMMs that contract over tokens or over d_out read the same row-major tensors
// "transposed"), selected in the shared-memory and instruction descriptors; nothing is
// transposed in memory.  Ragged sizes rely on TMA zero fill for loads, TMA clipping for stores
// and guarded per-thread stores.
//
// Every wait on an mbarrier is bounded: if it gives up, the kernel records FLOP_ERR_TIMEOUT,
// all roles leave their loops, outstanding copies are waited for (bounded), tensor memory is
// freed and the CTA returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace flop {
namespace tc {

constexpr int BM = 128;          // rows of D per tile = TMEM lanes
constexpr int BK = 64;           // K per stage = one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int kEpiWarps = 8;                 // two warps per TMEM lane quarter, each takes every other 32-column chunk
constexpr int kThreads = 64 + 32 * kEpiWarps;  // warp 0: TMA, warp 1: MMA, warps 2..9: epilogue
constexpr int kMaxStages = 8;
constexpr uint32_t kATileBytes = BM * BK * 2;     // 16 KB
constexpr uint32_t kBoxMN = 64;                   // MN-major operands arrive in 64(mn) x 64(k) boxes
constexpr uint32_t kBoxBytes = kBoxMN * BK * 2;   // 8 KB
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 2000000000LL;   // ~1 s
constexpr uint32_t kStoreBufBytes = 32 * 128;      // one epilogue warp's staging tile: 32 rows x 64 bf16

// Links between the problems of a chained launch (gemm_tc2_chain.cuh); all-zero for every other launch.
struct ChainLink {
  // producing side: every epilogue warp adds 1 to sig[tm] (tm = 256-row block) once its part of the tile is written
  unsigned* sig;
  // consuming side: the TMA producer waits until dep[row block] has 16 arrivals per N tile of the producing
  // problem.  dep_mode 1: the A operand is row block tm of that output; 2: the contraction runs over its rows.
  const unsigned* dep; int dep_mode;
  int dep_n_cap, dep_bn; const int* dep_dyn_n;     // N, N tile and device-side N (nullable) of the producing problem
  int side_dep;                                     // 1: the B operand is the diag(z) Q this launch forms as side work
  // side work asked for by this problem: sw_qz[k, :] = sw_z[k] * sw_q[k, :]  (sw_rows x sw_cols, bf16)
  const __nv_bfloat16* sw_q; int64_t sw_ldq; __nv_bfloat16* sw_qz; int64_t sw_ldqz; const float* sw_z; int sw_rows, sw_cols;
  // second stage of dlog_alpha inside the launch: fin[(tm*2 + cta)*4 + lane quarter] counts the N tiles of a 32-row
  // slab; the last arrival writes dla[row] (=|+=) dz_dla[row] * sum of the slab's partial row dots
  unsigned* fin; const float* dz_dla; float* dla; int dla_accumulate;
};

struct Params {
  int M, N, K;
  int bn;                 // N per tile: 64, 128, 192, 208 (CTA pairs, K-major B) or 256
  int stages;
  int tiles_m, tiles_n, splits, kb_per_split, num_kb;
  // floor(2^32 / d) + 1 for d = tiles_n and d = tiles_m * tiles_n: n / d == __umulhi(n, magic) for n, d < 65536
  // (div_fast = 1 when the problem has fewer than 65536 work items); saves the two integer divisions per tile decode
  uint32_t magic_tn, magic_tiles; int div_fast;
  // EPI_STORE: out[m*ldo + n] = acc * col_scale[n]  (bf16)
  __nv_bfloat16* out; int64_t ldo;
  const float* col_scale;               // nullable
  // EPI_SLICE: slices[split][m*ld_slice + n] = acc (fp32); optional fused row dot
  float* slices; int64_t slice_elems; int64_t ld_slice;
  const __nv_bfloat16* qdot; int64_t ldq;      // nullable: dz_part[(split*tiles_n+tn)*dz_stride + m] = sum_n acc*qdot[m,n]
  float* dz_part; int64_t dz_stride;
  int* dz_meta;                                // nullable: receives the number of partial vectors, 2 * tiles_n * splits
  // EPI_WGRAD (splits == 1): wg_out[m*ldo + n] (=|+=) row_scale[m] * acc, bf16 or fp32; same fused row dot
  void* wg_out; int wg_f32; const float* row_scale; int accumulate;
  int tma_store;   // 1: bf16 output tiles leave through shared memory and a TMA store (tensor map given)
  // Sizes known only on the device (nullable): the effective M, N, K are min(capacity, *ptr).  Used when the
  // rank dimension is the number of active components of a sampled mask.  Tiles outside the effective
  // extent are skipped by every role; the K loop stops at the 64-block that holds the last effective k, and
  // the N extent is rounded up to 64, so operands must be zero between the effective size and the next
  // multiple of 64.  An effective size of 0 is treated as 1 (an all-zero block).
  const int* dyn_m; const int* dyn_n; const int* dyn_k;
  int kind;   // 0 or 1: which of the two compile-time configurations of gemm2_dual_kernel serves this problem
  ChainLink link;
};

enum { EPI_STORE = 0, EPI_SLICE = 1, EPI_WGRAD = 2 };

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and records the timeout) if the phase never completes
// or another role has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
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

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the staging buffer may be overwritten once the earlier stores have read it
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (tcgen05): start address, leading/stride byte
// offsets (all >> 4), descriptor version 1, 128-byte swizzle.
//   K-major tile  (rows of 128 B = 64 bf16 along K): 8-row groups 1024 B apart (SBO); LBO unused.
//   MN-major tile (rows of 128 B = 64 bf16 along M/N, one row per k): 8-k groups 1024 B apart (SBO),
//                 successive 64-wide M/N chunks one box (8 KB) apart (LBO).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, bool mn_major) {
  const uint64_t lbo = mn_major ? (kBoxBytes >> 4) : 1;
  const uint64_t sbo = 1024 >> 4;
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, majors, N>>3, M>>4.
__device__ __forceinline__ uint32_t instr_desc(bool a_mn, bool b_mn, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__host__ __device__ inline uint32_t stage_bytes(int bn) { return kATileBytes + (uint32_t)bn * BK * 2; }
// tensor-memory columns between the two accumulator buffers (a multiple of 64; 2 x 256 is all there is)
__host__ __device__ inline uint32_t acc_stride(int bn_max) { return (uint32_t)((bn_max + 63) & ~63); }
// shared memory after the stage ring: the epilogue warps' staging tiles, then the barriers
constexpr uint32_t kStoreBufTotal = kEpiWarps * kStoreBufBytes;

struct WorkItem { int tm, tn, split, kb0, kb1; };
__device__ __forceinline__ WorkItem decode(const Params& p, int w) {
  WorkItem it;
  const int tiles = p.tiles_m * p.tiles_n;
  if (p.div_fast) {
    it.split = tiles == 1 ? w : (int)__umulhi((uint32_t)w, p.magic_tiles);
    const int t = w - it.split * tiles;
    it.tm = p.tiles_n == 1 ? t : (int)__umulhi((uint32_t)t, p.magic_tn);
    it.tn = t - it.tm * p.tiles_n;
  } else {
    it.split = w / tiles;
    const int t = w - it.split * tiles;
    it.tm = t / p.tiles_n;
    it.tn = t - it.tm * p.tiles_n;
  }
  it.kb0 = it.split * p.kb_per_split;
  it.kb1 = min(it.kb0 + p.kb_per_split, p.num_kb);
  return it;
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever arrives on, with the
// given cycle limit, and must come back with the timeout recorded (the status word is then read by
// flop_device_status()).  Exercises the exact wait routine of the GEMM kernels without a GEMM.
__global__ void wait_selftest_kernel(long long limit_cycles, int* gave_up) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint32_t b = smem_u32(&bar);
    const long long t0 = clock64();
    bool done = false;
    while (!done) {                       // the body of mbar_wait with a caller-chosen limit
      if (mbar_try_wait(b, 0)) break;
      if (clock64() - t0 > limit_cycles) {
        s_abort = 1;
        report_timeout();
        done = true;
      }
    }
    *gave_up = s_abort;
  }
}

// One 32-column chunk of one accumulator row (held by this thread) through the epilogue.
// n_end: first column that is not this tile's (the tile's end or the matrix's, whichever comes first).
template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const Params& p, uint32_t (&v)[32], int row, bool row_ok, int n0, int split,
                                               float& dot, int n_end) {
    const bool full_chunk = n0 + 32 <= n_end;
    if (EPI == EPI_STORE) {
      if (row_ok) {
        __nv_bfloat16* o = p.out + (int64_t)row * p.ldo + n0;
        if (full_chunk) {
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float a = __uint_as_float(v[2 * i]), b = __uint_as_float(v[2 * i + 1]);
            if (p.col_scale) { a *= __ldg(p.col_scale + n0 + 2 * i); b *= __ldg(p.col_scale + n0 + 2 * i + 1); }
            __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
            packed[i] = *reinterpret_cast<uint32_t*>(&h);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(o + 8 * i) = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
        } else {
          // ragged chunk: whole 8-column pieces as 16-byte stores (the tail of a 208-column tile is two of them),
          // the rest element by element
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (n0 + 8 * i + 8 <= n_end) {
              uint32_t pk[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                float a = __uint_as_float(v[8 * i + 2 * e]), b = __uint_as_float(v[8 * i + 2 * e + 1]);
                if (p.col_scale) { a *= __ldg(p.col_scale + n0 + 8 * i + 2 * e); b *= __ldg(p.col_scale + n0 + 8 * i + 2 * e + 1); }
                __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                pk[e] = *reinterpret_cast<uint32_t*>(&h);
              }
              *reinterpret_cast<uint4*>(o + 8 * i) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                if (n0 + 8 * i + e < n_end) {
                  float a = __uint_as_float(v[8 * i + e]);
                  if (p.col_scale) a *= __ldg(p.col_scale + n0 + 8 * i + e);
                  o[8 * i + e] = __float2bfloat16_rn(a);
                }
              }
            }
          }
        }
      }
    } else if (EPI == EPI_SLICE) {
      if (row_ok) {
        float* o = p.slices + (int64_t)split * p.slice_elems + (int64_t)row * p.ld_slice + n0;
        if (full_chunk) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4*>(o + 4 * i) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (n0 + i < n_end) o[i] = __uint_as_float(v[i]);
        }
        if (p.qdot) {
          const __nv_bfloat16* qr = p.qdot + (int64_t)row * p.ldq + n0;
          if (full_chunk) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint4 raw = __ldg(reinterpret_cast<const uint4*>(qr + 8 * i));
              const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(h[j]);
                dot = fmaf(__uint_as_float(v[8 * i + 2 * j]), f.x, dot);
                dot = fmaf(__uint_as_float(v[8 * i + 2 * j + 1]), f.y, dot);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < n_end) dot = fmaf(__uint_as_float(v[i]), __bfloat162float(qr[i]), dot);
          }
        }
      }
    } else {
      // weight gradient written in place: the fused row dot uses the unscaled accumulator, the
      // stored value carries the gate of this row (dQ = diag(z) M) and the caller's accumulate flag
      if (row_ok) {
        if (p.qdot) {
          const __nv_bfloat16* qr = p.qdot + (int64_t)row * p.ldq + n0;
          if (full_chunk) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint4 raw = __ldg(reinterpret_cast<const uint4*>(qr + 8 * i));
              const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(h[j]);
                dot = fmaf(__uint_as_float(v[8 * i + 2 * j]), f.x, dot);
                dot = fmaf(__uint_as_float(v[8 * i + 2 * j + 1]), f.y, dot);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < n_end) dot = fmaf(__uint_as_float(v[i]), __bfloat162float(qr[i]), dot);
          }
        }
        const float rs = p.row_scale ? __ldg(p.row_scale + row) : 1.f;
        if (p.wg_f32) {
          float* o = reinterpret_cast<float*>(p.wg_out) + (int64_t)row * p.ldo + n0;
          if (full_chunk) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float4 w = make_float4(__uint_as_float(v[4 * i]) * rs, __uint_as_float(v[4 * i + 1]) * rs,
                                     __uint_as_float(v[4 * i + 2]) * rs, __uint_as_float(v[4 * i + 3]) * rs);
              if (p.accumulate) {
                const float4 c = *reinterpret_cast<const float4*>(o + 4 * i);
                w.x += c.x; w.y += c.y; w.z += c.z; w.w += c.w;
              }
              *reinterpret_cast<float4*>(o + 4 * i) = w;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < n_end) o[i] = (p.accumulate ? o[i] : 0.f) + __uint_as_float(v[i]) * rs;
          }
        } else {
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.wg_out) + (int64_t)row * p.ldo + n0;
          if (full_chunk) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float w[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) w[j] = __uint_as_float(v[8 * i + j]) * rs;
              if (p.accumulate) {
                const uint4 c = *reinterpret_cast<const uint4*>(o + 8 * i);
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const float2 f = __bfloat1622float2(h[j]);
                  w[2 * j] += f.x; w[2 * j + 1] += f.y;
                }
              }
              uint32_t pk[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 hh = __floats2bfloat162_rn(w[2 * j], w[2 * j + 1]);
                pk[j] = *reinterpret_cast<uint32_t*>(&hh);
              }
              *reinterpret_cast<uint4*>(o + 8 * i) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < n_end)
                o[i] = __float2bfloat16_rn((p.accumulate ? __bfloat162float(o[i]) : 0.f) + __uint_as_float(v[i]) * rs);
          }
        }
      }
    }
}

// The row dot product <Q[row, n0..n0+31], acc> of the fused dz reduction, for the TMA-store path
// (the other paths compute it inside epilogue_chunk).
__device__ __forceinline__ void qdot_chunk(const Params& p, const uint32_t (&v)[32], int row, int n0, float& dot, int n_end) {
  const __nv_bfloat16* qr = p.qdot + (int64_t)row * p.ldq + n0;
  if (n0 + 32 <= n_end) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(qr + 8 * i));
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(h[j]);
        dot = fmaf(__uint_as_float(v[8 * i + 2 * j]), f.x, dot);
        dot = fmaf(__uint_as_float(v[8 * i + 2 * j + 1]), f.y, dot);
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (n0 + i < n_end) dot = fmaf(__uint_as_float(v[i]), __bfloat162float(qr[i]), dot);
  }
}

// Converts one 32-column chunk of this thread's accumulator row to bf16 (times the column gate
// or the row gate) and writes it as four 16-byte pieces into the warp's staging tile, laid out
// as the 128-byte-swizzled box the TMA store expects: row = lane, piece c at (c ^ (lane & 7)).
template <int EPI>
__device__ __forceinline__ void stage_chunk(const Params& p, const uint32_t (&v)[32], int row, int n0, uint32_t buf,
                                            int piece0, int lane) {
  const uint32_t row_addr = buf + (uint32_t)lane * 128u;
  const bool col_gate = EPI == EPI_STORE && p.col_scale;
  const bool row_gate = EPI == EPI_WGRAD && p.row_scale;
  if (!col_gate && !row_gate) {      // plain conversion
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t pk[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * j]), __uint_as_float(v[8 * i + 2 * j + 1]));
        pk[j] = *reinterpret_cast<uint32_t*>(&h);
      }
      st_shared_v4(row_addr + (uint32_t)(((piece0 + i) ^ (lane & 7)) << 4), pk[0], pk[1], pk[2], pk[3]);
    }
    return;
  }
  float sc[32];
  if (col_gate) {
    if (n0 + 32 <= p.N && (reinterpret_cast<uintptr_t>(p.col_scale + n0) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 f = __ldg(reinterpret_cast<const float4*>(p.col_scale + n0) + i);
        sc[4 * i] = f.x; sc[4 * i + 1] = f.y; sc[4 * i + 2] = f.z; sc[4 * i + 3] = f.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) sc[i] = n0 + i < p.N ? __ldg(p.col_scale + n0 + i) : 0.f;
    }
  } else {
    const float rs = row < p.M ? __ldg(p.row_scale + row) : 1.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) sc[i] = rs;
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * j]) * sc[8 * i + 2 * j],
                                               __uint_as_float(v[8 * i + 2 * j + 1]) * sc[8 * i + 2 * j + 1]);
      pk[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    st_shared_v4(row_addr + (uint32_t)(((piece0 + i) ^ (lane & 7)) << 4), pk[0], pk[1], pk[2], pk[3]);
  }
}

// Epilogue of one accumulator tile for one epilogue warp.  Lane quarter q = warp & 3 fixes the
// 32 accumulator rows this warp may read; h = 0/1 picks the even or odd 64-column groups.  A group
// (two 32-column chunks) is fetched from tensor memory per wait, and the accumulator is handed back
// to the MMA warp (arrive on `release_bar`, a CTA-local or cluster address) as soon as the last
// fetch has landed in registers, before conversion and stores.
// Output path: with p.tma_store the 32 x 64 bf16 block is staged in shared memory (`store_buf`,
// this warp's 4 KB) and leaves with one TMA store -- a thread owns a ROW of the accumulator, so
// direct global stores would touch 32 different rows per instruction (32 partial sectors), which
// measured ~7000 cycles per block against the ~400 of the staged store; the tensor map also clips
// the ragged edges.  Otherwise (fp32 outputs, accumulate, split-K slices) each thread stores its row.
// Arrival on a barrier that may live in the other CTA of the pair.  CTA-scope release: the tensor-memory loads this
// arrival hands back are complete (tcgen05.wait::ld) and fenced (tcgen05.fence::before_thread_sync) when it is
// issued, and the thread publishes no ordinary memory with it.  A cluster-scope release here made the thread wait for
// all its outstanding stores to be acknowledged, 1000-1500 cycles per tile under load.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}

template <int EPI, bool kClusterArrive>
__device__ __forceinline__ void run_epilogue(const Params& p, const CUtensorMap* tmap_out, uint32_t store_buf, uint32_t t_acc,
                                             int row0, int n_base, int n_limit, int split, int tn, int warp, int lane,
                                             uint32_t release_bar) {
  const int q = warp & 3, h = (warp - 2) >> 2;
  const int row = row0 + q * 32 + lane;
  const bool row_ok = row < p.M;
  const uint32_t t_row = t_acc + ((uint32_t)(q * 32) << 16);
  const int nchunks = (min(p.bn, n_limit - n_base) + 31) >> 5;   // 32-column chunks that hold columns of D
  const int ngroups = (nchunks + 1) >> 1;                    // 64-column groups
  // An N tile that is not a multiple of 64 columns wide (208) ends inside its last group: the staged 64-column
  // store would run into the next tile, so that group is written by per-thread stores masked at the tile's end
  // (at the matrix's edge the tensor map clips, as for every tile).
  const int tile_end = min(n_base + p.bn, p.N);
  float dot = 0.f;
  bool released = false;
  for (int g = h; g < ngroups; g += 2) {
    const int c0 = 2 * g, c1 = c0 + 1;
    const bool two = c1 < nchunks;
    uint32_t v0[32], v1[32];
    tmem_ld32(t_row + (uint32_t)(c0 * 32), v0);
    if (two) tmem_ld32(t_row + (uint32_t)(c1 * 32), v1);
    tmem_ld_wait();
    if (g + 2 >= ngroups) {
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kClusterArrive) mbar_arrive_remote(release_bar);
        else mbar_arrive(release_bar);
      }
      released = true;
    }
    const int n0 = n_base + c0 * 32;
    if (p.tma_store && !(n0 + 64 > tile_end && tile_end < p.N)) {
      if (EPI != EPI_STORE && p.qdot && row_ok) {
        qdot_chunk(p, v0, row, n0, dot, tile_end);
        if (two) qdot_chunk(p, v1, row, n0 + 32, dot, tile_end);
      }
      if (lane == 0) tma_store_wait_read();   // the previous block has left the staging tile
      __syncwarp();
      stage_chunk<EPI>(p, v0, row, n0, store_buf, 0, lane);
      if (two) stage_chunk<EPI>(p, v1, row, n0 + 32, store_buf, 4, lane);
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && row0 + q * 32 < p.M) tma_store_2d(tmap_out, n0, row0 + q * 32, store_buf);   // never start a store outside the tensor
    } else {
      epilogue_chunk<EPI>(p, v0, row, row_ok, n0, split, dot, tile_end);
      if (two) epilogue_chunk<EPI>(p, v1, row, row_ok, n0 + 32, split, dot, tile_end);
    }
  }
  if (!released) {   // this warp had no group in the tile
    tcgen05_fence_before();
    __syncwarp();
    if (lane == 0) {
      if (kClusterArrive) mbar_arrive_remote(release_bar);
      else mbar_arrive(release_bar);
    }
  }
  if (EPI != EPI_STORE && p.qdot && row_ok) {
    p.dz_part[(int64_t)((split * p.tiles_n + tn) * 2 + h) * p.dz_stride + row] = dot;
    if (p.dz_meta && row == 0 && tn == 0 && split == 0 && h == 0) *p.dz_meta = 2 * p.tiles_n * p.splits;
  }
}

}  // namespace tc
}  // namespace flop
