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
        if (tid == 0) {
          int acc = 0, b = 255;
          for (; b > 0; --b) {
            if (acc + hist[b] >= need) break;
            acc += hist[b];
          }
          s_prefix = prefix | ((uint32_t)b << shift);
          s_need = need - acc;
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

}  // namespace flop
