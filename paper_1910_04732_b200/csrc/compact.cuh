// Deterministic inference mask and rank compaction (Sections 4.4 and 4.1).
//
//   compact_select_kernel : one block.  mode 0: pi_j in fp64, k = floor(sum pi + 1/2),
//       exact top-k of log_alpha by a 4-pass radix select on order-preserving
//       keys (ties -> lower index), then a block scan (warp shuffles) that
//       writes the ascending index list.  mode 1: keep z_j > 0.
//   gather_q_kernel : Qc[c, :] = z[idx[c]] * Q[idx[c], :]   (row gather, 16-byte vectors)
//   gather_p_kernel : Pc[i, c] = P[i, idx[c]]  (each P row is read once, coalesced,
//       into shared memory and the surviving columns are written out coalesced)
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float a) {
  a += 0.0f;  // -0 -> +0 so that equal values have equal keys
  const uint32_t b = __float_as_uint(a);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kSelThreads)
compact_select_kernel(const float* __restrict__ in, int mode, double thr, int r, int32_t* __restrict__ idx,
                      int32_t* __restrict__ k_dev, float* __restrict__ z_det) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ double red[32];
  __shared__ int hist[256];
  __shared__ int scan_scratch[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  const int tid = threadIdx.x;
  int k = 0;
  uint32_t kth = 0;   // key of the k-th largest gate
  int need_eq = 0;    // how many gates with key == kth are kept (lowest indices first)
  if (mode == 0) {
    double sum = 0.0;
    for (int j = tid; j < r; j += kSelThreads) sum += 1.0 / (1.0 + exp(-((double)in[j] - thr)));
    sum = block_sum_f64(sum, red);
    k = (int)floor(sum + 0.5);
    k = max(0, min(r, k));
    if (k > 0) {
      // radix select, most significant byte first
      uint32_t prefix = 0, pmask = 0;
      int need = k;   // rank (1-based, from the top) still to be located inside the prefix class
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < r; j += kSelThreads) {
          const uint32_t key = order_key(in[j]);
          if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        {
          // the bin that holds the need-th largest key: a block scan over the bins from the top (thread t holds bin
          // 255 - t), instead of one thread walking 256 counters
          const int h = tid < 256 ? hist[255 - tid] : 0;
          int tot = 0;
          const int above = block_exclusive_scan(h, scan_scratch, &tot);
          if (tid < 256 && above < need && need <= above + h) {
            s_prefix = prefix | ((uint32_t)(255 - tid) << shift);
            s_need = need - above;
          }
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        pmask |= 255u << shift;
        __syncthreads();
      }
      kth = prefix;
      need_eq = need;
    }
  }
  // ordered scan over the gates: running count of kept gates and of ties seen
  int base_keep = 0, base_eq = 0;
  for (int j0 = 0; j0 < r; j0 += kSelThreads) {
    const int j = j0 + tid;
    float v = 0.f;
    int eq = 0, gt = 0;
    if (j < r) {
      v = in[j];
      if (mode == 0) {
        const uint32_t key = order_key(v);
        gt = (k > 0) && key > kth;
        eq = (k > 0) && key == kth;
      } else {
        gt = v > 0.f;
      }
    }
    int tot_eq = 0, tot_keep = 0;
    const int rank_eq = mode == 0 ? base_eq + block_exclusive_scan(eq, scan_scratch, &tot_eq) : 0;
    const int keep = gt || (eq && rank_eq < need_eq);
    const int pos = base_keep + block_exclusive_scan(keep, scan_scratch, &tot_keep);
    if (j < r) {
      if (keep) idx[pos] = j;
      if (z_det) {
        float zv = 0.f;
        if (keep) zv = mode == 0 ? (float)(1.0 / (1.0 + exp(-((double)v - thr)))) : v;
        z_det[j] = zv;
      }
    }
    base_eq += tot_eq;
    base_keep += tot_keep;
  }
  if (tid == 0) *k_dev = base_keep;
}

// 16-byte vector of elements
template <typename T> struct Vec16 { static constexpr int n = 16 / sizeof(T); };

template <typename T>
__global__ void __launch_bounds__(256)
gather_q_kernel(const T* __restrict__ Q, int64_t ldq, const int32_t* __restrict__ idx, const int32_t* __restrict__ k_dev,
                const float* __restrict__ z, int d_in, T* __restrict__ Qc, int64_t ldqc, int vec_ok) {
  pdl_wait();
  pdl_launch_dependents();
  const int c = blockIdx.x;
  if (c >= *k_dev) return;
  const int src = idx[c];
  const float g = z[src];
  const T* q = Q + (int64_t)src * ldq;
  T* o = Qc + (int64_t)c * ldqc;
  constexpr int V = Vec16<T>::n;
  if (vec_ok) {
    for (int j = threadIdx.x * V; j < d_in; j += blockDim.x * V) {
      if (j + V <= d_in) {
        uint4 raw = *reinterpret_cast<const uint4*>(q + j);
        T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
        for (int i = 0; i < V; ++i) e[i] = from_f32<T>(to_f32<T>(e[i]) * g);
        *reinterpret_cast<uint4*>(o + j) = raw;
      } else {
        for (int i = j; i < d_in; ++i) o[i] = from_f32<T>(to_f32<T>(q[i]) * g);
      }
    }
  } else {
    for (int j = threadIdx.x; j < d_in; j += blockDim.x) o[j] = from_f32<T>(to_f32<T>(q[j]) * g);
  }
}

// One block per kRows rows of P; a row (r elements) is staged in shared memory.
template <typename T>
__global__ void __launch_bounds__(256)
gather_p_kernel(const T* __restrict__ P, int64_t ldp, const int32_t* __restrict__ idx, const int32_t* __restrict__ k_dev,
                int r, int d_out, T* __restrict__ Pc, int64_t ldpc, int rows_per_block, int vec_ok) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* row = reinterpret_cast<T*>(smem_raw);
  const int k = *k_dev;
  constexpr int V = Vec16<T>::n;
  for (int rr = 0; rr < rows_per_block; ++rr) {
    const int i = blockIdx.x * rows_per_block + rr;
    if (i >= d_out) return;
    const T* p = P + (int64_t)i * ldp;
    if (vec_ok) {
      for (int j = threadIdx.x * V; j < r; j += blockDim.x * V) {
        if (j + V <= r) *reinterpret_cast<uint4*>(row + j) = *reinterpret_cast<const uint4*>(p + j);
        else for (int e = j; e < r; ++e) row[e] = p[e];
      }
    } else {
      for (int j = threadIdx.x; j < r; j += blockDim.x) row[j] = p[j];
    }
    __syncthreads();
    T* o = Pc + (int64_t)i * ldpc;
    // four surviving columns per thread and store where the element type and the alignment allow it
    // (8-byte stores, 256 bytes per warp instruction), single elements otherwise
    if (sizeof(T) == 2 && (reinterpret_cast<uintptr_t>(o) & 7) == 0 && (reinterpret_cast<uintptr_t>(idx) & 15) == 0) {
      for (int c = threadIdx.x * 4; c < k; c += blockDim.x * 4) {
        if (c + 3 < k) {
          const int4 ii = *reinterpret_cast<const int4*>(idx + c);
          T quad[4] = {row[ii.x], row[ii.y], row[ii.z], row[ii.w]};
          *reinterpret_cast<uint2*>(o + c) = *reinterpret_cast<uint2*>(quad);
        } else {
          for (int e = c; e < k; ++e) o[e] = row[idx[e]];
        }
      }
    } else {
      for (int c = threadIdx.x; c < k; c += blockDim.x) o[c] = row[idx[c]];
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// P gather with the rows staged by bulk asynchronous copies (bf16, rows of a multiple of 16 bytes).
//
// A block walks groups of `rows_per_stage` consecutive rows of P.  One thread hands the rows of the
// next groups to the copy engine (cp.async.bulk global -> shared, completion counted in bytes on an
// mbarrier per buffer) while all threads pick the surviving columns of the current group out of
// shared memory and write them as 8-byte pieces, so the read of P is fully coalesced, needs no
// registers or load instructions, and overlaps the select/store phase of the same block.  The
// index list is kept in shared memory as 16-bit entries (r <= 65536).  Waits are bounded: when one
// gives up, the block records FLOP_ERR_TIMEOUT, lets the copies in flight land (bounded) and returns.
namespace gp {
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// 16-byte aligned source and destination, size a multiple of 16 bytes
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
constexpr long long kWaitCycles = 2000000000LL;   // ~1 s
}  // namespace gp

constexpr int kGatherMaxBuf = 4;

__global__ void __launch_bounds__(256)
gather_p_pipe_kernel(const __nv_bfloat16* __restrict__ P, int64_t ldp, const int32_t* __restrict__ idx,
                     const int32_t* __restrict__ k_dev, int r, int d_out, __nv_bfloat16* __restrict__ Pc, int64_t ldpc,
                     int rows_per_stage, int nbuf) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];   // every offset used below is a multiple of 16
  __shared__ int s_abort;
  const int k = min(*k_dev, r);
  if (k <= 0) return;
  const uint32_t row_bytes = (uint32_t)r * 2u;                     // multiple of 16 (checked by the host)
  const uint32_t stage_bytes = row_bytes * (uint32_t)rows_per_stage;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw);            // nbuf barriers (64 bytes reserved)
  unsigned short* sidx = reinterpret_cast<unsigned short*>(smem_raw + 64);               // r entries
  unsigned char* bufs = smem_raw + 64 + (((size_t)r * 2 + 127) & ~(size_t)127);          // nbuf stages
  const int n_groups = (d_out + rows_per_stage - 1) / rows_per_stage;
  const int n_mine = (int)blockIdx.x < n_groups ? (n_groups - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  if (n_mine == 0) return;

  auto issue = [&](int it) {   // thread 0: hand the rows of this block's it-th group to the copy engine
    const int b = it % nbuf;
    const int row0 = ((int)blockIdx.x + it * (int)gridDim.x) * rows_per_stage;
    const int rows = min(rows_per_stage, d_out - row0);
    const uint32_t bar = gp::smem_addr(&bars[b]);
    gp::bar_expect_tx(bar, row_bytes * (uint32_t)rows);
    for (int j = 0; j < rows; ++j)
      gp::bulk_load(gp::smem_addr(bufs + (size_t)b * stage_bytes + (size_t)j * row_bytes), P + (int64_t)(row0 + j) * ldp, row_bytes, bar);
  };

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int b = 0; b < nbuf; ++b) gp::bar_init(gp::smem_addr(&bars[b]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int it = 0; it < min(nbuf, n_mine); ++it) issue(it);
  }
  for (int c = threadIdx.x; c < k; c += blockDim.x) sidx[c] = (unsigned short)idx[c];
  __syncthreads();

  const int kq = (k + 3) >> 2;   // 4-column pieces per row
  const bool vec_out = (reinterpret_cast<uintptr_t>(Pc) & 7) == 0 && (ldpc & 3) == 0;
  int issued = min(nbuf, n_mine);
  for (int it = 0; it < n_mine; ++it) {
    const int b = it % nbuf;
    const uint32_t parity = (uint32_t)(it / nbuf) & 1u;
    const uint32_t bar = gp::smem_addr(&bars[b]);
    if (!gp::bar_try_wait(bar, parity)) {
      const long long t0 = clock64();
      while (!gp::bar_try_wait(bar, parity)) {
        if (*(volatile int*)&s_abort) break;
        if (clock64() - t0 > gp::kWaitCycles) { *(volatile int*)&s_abort = 1; report_timeout(); break; }
      }
    }
    if (__syncthreads_or(s_abort)) break;   // every thread takes the same decision
    const int row0 = ((int)blockIdx.x + it * (int)gridDim.x) * rows_per_stage;
    const int rows = min(rows_per_stage, d_out - row0);
    const __nv_bfloat16* stage = reinterpret_cast<const __nv_bfloat16*>(bufs + (size_t)b * stage_bytes);
    for (int w = threadIdx.x; w < rows * kq; w += blockDim.x) {
      const int j = w / kq, c = (w - j * kq) << 2;
      const __nv_bfloat16* row = stage + (size_t)j * r;
      __nv_bfloat16* o = Pc + (int64_t)(row0 + j) * ldpc + c;
      if (c + 3 < k && vec_out) {
        const uint2 ii = *reinterpret_cast<const uint2*>(sidx + c);   // four 16-bit indices
        const unsigned short q0 = __bfloat16_as_ushort(row[ii.x & 0xFFFFu]), q1 = __bfloat16_as_ushort(row[ii.x >> 16]);
        const unsigned short q2 = __bfloat16_as_ushort(row[ii.y & 0xFFFFu]), q3 = __bfloat16_as_ushort(row[ii.y >> 16]);
        __stcs(reinterpret_cast<uint2*>(o), make_uint2((uint32_t)q0 | ((uint32_t)q1 << 16), (uint32_t)q2 | ((uint32_t)q3 << 16)));
      } else {
        for (int e = c; e < min(c + 4, k); ++e) o[e - c] = row[sidx[e]];
      }
    }
    __syncthreads();   // the buffer has been read by everyone: it may be refilled
    if (threadIdx.x == 0 && issued < n_mine) issue(issued);
    if (issued < n_mine) ++issued;
  }
  if (s_abort && threadIdx.x == 0) {
    // leaving early: give the copies already issued time to land so that nothing writes this block's
    // shared memory after it has gone
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}
  }
}

}  // namespace flop
