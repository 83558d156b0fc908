// Training on the active rank components only.
//
// The gate sample z is shared by the whole batch, so components with z_k = 0 contribute nothing
// to this step's forward or backward pass; the paper selects "the parameters that are only active
// for the current batch" and runs smaller matrix products (Section 4.3, last paragraph).  Three
// grouped kernels (blockIdx.y = matrix of the group) do the selection and the data movement; the
// GEMMs then run on the compact factors with the rank read from device memory:
//   active_select_kernel   idx = {k : z_k > 0} ascending, pos = inverse map, k_dev, and the compact
//                          gate vectors z_c = z[idx], dz_dla_c = dz_dla[idx] (zero beyond k)
//   active_gather_kernel   Q_c[c,:] = Q[idx[c],:] (UNscaled: the gate stays in the GEMM epilogue and
//                          the fused <Q, .> reduction needs the raw rows), P_c[:,c] = P[:,idx[c]];
//                          rows / columns from k up to the next multiple of 64 are zero-filled,
//                          because the GEMMs' K loops and N extents run to that boundary; optionally
//                          also Qz_c = diag(z_c) Q_c, the backward pass's B operand for dX
//   active_scatter_kernel  dP[:,idx] = dP_c, dQ[idx,:] = dQ_c, dlog_alpha[idx] = dlog_alpha_c and
//                          exact zeros everywhere else (or += when accumulating)
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kActiveGroup = 96;   // matrices per launch: a whole model's worth in one group (argument block ~13 KB)

struct ActiveGather {
  const float* z; const float* dz_dla;                 // [r], dz_dla nullable
  const __nv_bfloat16* P; int64_t ldp; const __nv_bfloat16* Q; int64_t ldq;
  int r, d_in, d_out;
  int32_t* idx; int32_t* pos; int32_t* k_dev;          // [r], [r], [1]
  float* z_c; float* dz_dla_c;                         // [r], dz_dla_c nullable
  __nv_bfloat16* P_c; int64_t ldpc; __nv_bfloat16* Q_c; int64_t ldqc;
  __nv_bfloat16* Qz_c; int64_t ldqzc;                  // nullable: diag(z_c) Q_c
};
struct ActiveGatherGroup { ActiveGather a[kActiveGroup]; int n; };

__global__ void __launch_bounds__(1024)
active_select_kernel(const __grid_constant__ ActiveGatherGroup g) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int scan_scratch[33];
  const ActiveGather& a = g.a[blockIdx.x];
  const int tid = threadIdx.x, r = a.r;
  int base = 0;
  for (int j0 = 0; j0 < r; j0 += 1024) {
    const int j = j0 + tid;
    const float v = j < r ? a.z[j] : 0.f;
    const int keep = v > 0.f;
    int tot = 0;
    const int p = base + block_exclusive_scan(keep, scan_scratch, &tot);
    if (j < r) {
      a.pos[j] = keep ? p : -1;
      if (keep) {
        a.idx[p] = j;
        a.z_c[p] = v;
        if (a.dz_dla_c) a.dz_dla_c[p] = a.dz_dla[j];
      }
    }
    base += tot;
  }
  for (int c = base + tid; c < r; c += 1024) {   // compact gates are zero beyond the active count
    a.z_c[c] = 0.f;
    if (a.dz_dla_c) a.dz_dla_c[c] = 0.f;
  }
  if (tid == 0) *a.k_dev = base;
}

__device__ __forceinline__ int pad64(int k) { return (max(k, 1) + 63) & ~63; }

constexpr int kActiveWarps = 8;   // one row task per warp, eight per block

// Row task t = blockIdx.x * 8 + warp: t < r is compact row t of Q_c, otherwise row t - r of P_c.
__global__ void __launch_bounds__(32 * kActiveWarps)
active_gather_kernel(const __grid_constant__ ActiveGatherGroup g, int smem_row_elems) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const ActiveGather& a = g.a[blockIdx.y];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kActiveWarps + warp;
  const int k = *a.k_dev, kp = min(a.r, pad64(k));
  if (t < a.r) {
    const int c = t;
    if (c >= kp) return;
    __nv_bfloat16* o = a.Q_c + (int64_t)c * a.ldqc;
    __nv_bfloat16* oz = a.Qz_c ? a.Qz_c + (int64_t)c * a.ldqzc : nullptr;
    if (c < k) {
      const int src = a.idx[c];
      const __nv_bfloat16* q = a.Q + (int64_t)src * a.ldq;
      const float zc = a.z[src];
      for (int j = lane * 8; j < a.d_in; j += 32 * 8) {     // rows are 16-byte aligned (ld % 8 == 0)
        if (j + 8 <= a.d_in) {
          const uint4 raw = *reinterpret_cast<const uint4*>(q + j);
          *reinterpret_cast<uint4*>(o + j) = raw;
          if (oz) {
            uint4 sc = raw;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&sc);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 x = __bfloat1622float2(h[e]);
              h[e] = __floats2bfloat162_rn(x.x * zc, x.y * zc);
            }
            *reinterpret_cast<uint4*>(oz + j) = sc;
          }
        } else {
          for (int e = j; e < a.d_in; ++e) {
            o[e] = q[e];
            if (oz) oz[e] = __float2bfloat16_rn(__bfloat162float(q[e]) * zc);
          }
        }
      }
    } else {
      for (int j = lane; j < a.d_in; j += 32) {
        o[j] = __float2bfloat16_rn(0.f);
        if (oz) oz[j] = __float2bfloat16_rn(0.f);
      }
    }
  } else {
    const int i = t - a.r;
    if (i >= a.d_out) return;
    __nv_bfloat16* row = reinterpret_cast<__nv_bfloat16*>(smem_raw) + (size_t)warp * smem_row_elems;
    const __nv_bfloat16* p = a.P + (int64_t)i * a.ldp;
    for (int j = lane * 8; j < a.r; j += 32 * 8) {
      if (j + 8 <= a.r) *reinterpret_cast<uint4*>(row + j) = *reinterpret_cast<const uint4*>(p + j);
      else for (int e = j; e < a.r; ++e) row[e] = p[e];
    }
    __syncwarp();
    __nv_bfloat16* o = a.P_c + (int64_t)i * a.ldpc;
    for (int c = lane; c < kp; c += 32) o[c] = c < k ? row[a.idx[c]] : __float2bfloat16_rn(0.f);
  }
}

struct ActiveScatter {
  const int32_t* idx; const int32_t* pos; const int32_t* k_dev;
  int r, d_in, d_out;
  const void* dP_c; int64_t lddpc; const void* dQ_c; int64_t lddqc; const float* dla_c;   // any may be null
  void* dP; int64_t lddp; void* dQ; int64_t lddq; float* dla;
};
struct ActiveScatterGroup { ActiveScatter a[kActiveGroup]; int n; int accumulate; };

// Row task t = blockIdx.x * 8 + warp: t < r is row t of dQ (and dlog_alpha[t]), otherwise row t - r of dP.
template <typename TW>
__global__ void __launch_bounds__(32 * kActiveWarps)
active_scatter_kernel(const __grid_constant__ ActiveScatterGroup g) {
  pdl_wait();
  pdl_launch_dependents();
  const ActiveScatter& a = g.a[blockIdx.y];
  const int acc = g.accumulate;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kActiveWarps + warp;
  if (t < a.r) {
    const int j = t;
    const int c = a.pos[j];
    if (a.dQ) {
      TW* o = reinterpret_cast<TW*>(a.dQ) + (int64_t)j * a.lddq;
      constexpr int V = 16 / (int)sizeof(TW);
      const TW* s = c >= 0 ? reinterpret_cast<const TW*>(a.dQ_c) + (int64_t)c * a.lddqc : nullptr;
      const bool vec = !acc && ((reinterpret_cast<uintptr_t>(o) | reinterpret_cast<uintptr_t>(s)) & 15) == 0;
      if (vec) {       // plain copy or zero fill, 16 bytes per lane
        for (int e = lane * V; e < a.d_in; e += 32 * V) {
          if (e + V <= a.d_in) *reinterpret_cast<uint4*>(o + e) = s ? *reinterpret_cast<const uint4*>(s + e) : make_uint4(0, 0, 0, 0);
          else for (int x = e; x < a.d_in; ++x) o[x] = s ? s[x] : from_f32<TW>(0.f);
        }
      } else if (c >= 0) {
        for (int e = lane; e < a.d_in; e += 32) o[e] = acc ? from_f32<TW>(to_f32<TW>(o[e]) + to_f32<TW>(s[e])) : s[e];
      } else if (!acc) {
        for (int e = lane; e < a.d_in; e += 32) o[e] = from_f32<TW>(0.f);
      }
    }
    if (a.dla && lane == 0) {
      const float v = c >= 0 ? a.dla_c[c] : 0.f;
      a.dla[j] = acc ? a.dla[j] + v : v;
    }
  } else {
    const int i = t - a.r;
    if (i >= a.d_out || !a.dP) return;
    TW* o = reinterpret_cast<TW*>(a.dP) + (int64_t)i * a.lddp;
    const TW* s = reinterpret_cast<const TW*>(a.dP_c) + (int64_t)i * a.lddpc;
    // coalesced row write, 16 bytes per lane; the read of dP_c is a gather within one (cached) row
    constexpr int V = 16 / (int)sizeof(TW);
    const bool vec = !acc && (reinterpret_cast<uintptr_t>(o) & 15) == 0;
    for (int j0 = lane * V; j0 < a.r; j0 += 32 * V) {
      if (vec && j0 + V <= a.r) {
        uint4 raw;
        TW* e = reinterpret_cast<TW*>(&raw);
#pragma unroll
        for (int x = 0; x < V; ++x) {
          const int c = __ldg(a.pos + j0 + x);
          e[x] = c >= 0 ? s[c] : from_f32<TW>(0.f);
        }
        *reinterpret_cast<uint4*>(o + j0) = raw;
      } else {
        for (int j = j0; j < min(j0 + V, a.r); ++j) {
          const int c = a.pos[j];
          const float v = c >= 0 ? to_f32<TW>(s[c]) : 0.f;
          o[j] = acc ? from_f32<TW>(to_f32<TW>(o[j]) + v) : from_f32<TW>(v);
        }
      }
    }
  }
}

}  // namespace flop
