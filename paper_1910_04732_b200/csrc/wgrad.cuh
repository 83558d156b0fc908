// Small kernels around the backward GEMMs: the ordered split-K reduction of the
// weight gradients with the gate epilogue, the dlog_alpha second stage, and
// the pre-scaled factor diag(z) Q used by dX.
#pragma once
#include "common.cuh"

namespace flop {

// Qz[k, :] = z[k] * Q[k, :]
template <typename T>
__global__ void __launch_bounds__(256)
scale_rows_kernel(const T* __restrict__ Q, int64_t ldq, const float* __restrict__ z, int rows, int cols,
                  T* __restrict__ out, int64_t ldo) {
  pdl_wait();
  pdl_launch_dependents();
  const int k = blockIdx.x;
  if (k >= rows) return;
  const float g = z[k];
  constexpr int V = 16 / sizeof(T);
  const T* q = Q + (int64_t)k * ldq;
  T* o = out + (int64_t)k * ldo;
  const bool vec = ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(o)) & 15) == 0;
  if (vec) {
    for (int j = threadIdx.x * V; j < cols; j += blockDim.x * V) {
      if (j + V <= cols) {
        uint4 raw = *reinterpret_cast<const uint4*>(q + j);
        T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
        for (int i = 0; i < V; ++i) e[i] = from_f32<T>(to_f32<T>(e[i]) * g);
        *reinterpret_cast<uint4*>(o + j) = raw;
      } else {
        for (int i = j; i < cols; ++i) o[i] = from_f32<T>(to_f32<T>(q[i]) * g);
      }
    }
  } else {
    for (int j = threadIdx.x; j < cols; j += blockDim.x) o[j] = from_f32<T>(to_f32<T>(q[j]) * g);
  }
}

// Weight-gradient finalisation.  slices[s][m][n] (fp32, ld = ld_slice, slice
// stride = slice_elems) are the split-K partial products, summed here in slice
// order (bit-reproducible).  out[m,n] (=|+=) row_scale[m] * sum.
// If qdot != nullptr, also dz_part[blockIdx.y-th column block][m] = sum_n Qdot[m,n] * sum (unscaled),
// one block row per m: a block handles one row m and strides over n.
template <typename TOut, typename TQ>
__global__ void __launch_bounds__(256)
wgrad_finalize_kernel(const float* __restrict__ slices, int n_slices, int64_t slice_elems, int64_t ld_slice,
                      int M, int N, const float* __restrict__ row_scale, TOut* __restrict__ out, int64_t ldo,
                      int accumulate, const TQ* __restrict__ qdot, int64_t ldq, float* __restrict__ dz_out) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ double red[32];
  const int m = blockIdx.x;
  if (m >= M) return;
  const float rs = row_scale ? row_scale[m] : 1.f;
  double dot = 0.0;
  for (int n = threadIdx.x; n < N; n += blockDim.x) {
    float v = 0.f;
    for (int s = 0; s < n_slices; ++s) v += slices[(int64_t)s * slice_elems + (int64_t)m * ld_slice + n];
    if (qdot) dot += (double)v * (double)to_f32<TQ>(qdot[(int64_t)m * ldq + n]);
    if (out) {
      TOut* o = out + (int64_t)m * ldo + n;
      const float w = v * rs;
      *o = from_f32<TOut>(accumulate ? to_f32<TOut>(*o) + w : w);
    }
  }
  if (qdot) {
    dot = block_sum_f64(dot, red);
    if (threadIdx.x == 0) dz_out[m] = (float)dot;
  }
}

// dlog_alpha[k] (=|+=) dz_dla[k] * sum_p dz_part[p][k], partials added in order.
__global__ void __launch_bounds__(256)
dalpha_kernel(const float* __restrict__ dz_part, int n_part, int64_t part_stride, const float* __restrict__ dz_dla,
              int r, float* __restrict__ dlog_alpha, int accumulate) {
  pdl_wait();
  pdl_launch_dependents();
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= r) return;
  float s = 0.f;
  for (int p = 0; p < n_part; ++p) s += dz_part[(int64_t)p * part_stride + k];
  const float v = s * dz_dla[k];
  dlog_alpha[k] = accumulate ? dlog_alpha[k] + v : v;
}


// One launch that finishes the backward pass of the tensor-core path:
//   dP[i,k]      (=|+=) sum_s slices_p[s][i,k]                      (d_out x r)
//   dQ[k,j]      (=|+=) z[k] * sum_s slices_q[s][k,j]               (r x d_in)
//   Qz[k,j]      =      z[k] * Q[k,j]                                (r x d_in, feeds the dX GEMM)
//   dlog_alpha[k](=|+=) dz_dla[k] * sum_p dz_part[p][k]
// Split-K slices and dz partials are added in index order (bit-reproducible).  Work is cut into
// units of 4 consecutive columns of one row; a grid-stride loop walks the four regions in turn.
struct BwdFinishArgs {
  const float* slices_p; int n_slices_p; int64_t slice_elems_p, ld_slice_p; int d_out, r;
  void* dP; int64_t lddp;
  const float* slices_q; int n_slices_q; int64_t slice_elems_q, ld_slice_q; int d_in;
  void* dQ; int64_t lddq;
  const float* z;
  const __nv_bfloat16* Q; int64_t ldq; __nv_bfloat16* Qz; int64_t ldqz;
  const float* dz_part; int n_part; const float* dz_dla; float* dlog_alpha;
  int accumulate;
};

template <typename TW>
__device__ __forceinline__ void store4(TW* o, const float (&v)[4], int valid, int accumulate, bool vec) {
  if (vec && valid == 4) {
    if constexpr (sizeof(TW) == 4) {
      float4 w = make_float4(v[0], v[1], v[2], v[3]);
      if (accumulate) { const float4 c = *reinterpret_cast<const float4*>(o); w.x += c.x; w.y += c.y; w.z += c.z; w.w += c.w; }
      *reinterpret_cast<float4*>(o) = w;
    } else {
      float w[4] = {v[0], v[1], v[2], v[3]};
      if (accumulate) {
        const uint2 c = *reinterpret_cast<const uint2*>(o);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&c);
        const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
        w[0] += a.x; w[1] += a.y; w[2] += b.x; w[3] += b.y;
      }
      __nv_bfloat162 lo = __floats2bfloat162_rn(w[0], w[1]), hi = __floats2bfloat162_rn(w[2], w[3]);
      uint2 out;
      out.x = *reinterpret_cast<uint32_t*>(&lo);
      out.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(o) = out;
    }
  } else {
    for (int i = 0; i < valid; ++i) o[i] = from_f32<TW>(accumulate ? to_f32<TW>(o[i]) + v[i] : v[i]);
  }
}

template <typename TW>
__device__ __forceinline__ void reduce_unit(const float* __restrict__ slices, int n_slices, int64_t slice_elems, int64_t ld_slice,
                                            int row, int c0, int ncols, float scale, TW* __restrict__ out, int64_t ldo,
                                            int accumulate, bool vec_out) {
  const int valid = min(4, ncols - c0);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  const float* src = slices + (int64_t)row * ld_slice + c0;
  if (valid == 4) {
    for (int s = 0; s < n_slices; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(src + (int64_t)s * slice_elems);
      acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
    }
  } else {
    for (int s = 0; s < n_slices; ++s)
      for (int i = 0; i < valid; ++i) acc[i] += src[(int64_t)s * slice_elems + i];
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) acc[i] *= scale;
  store4<TW>(out + (int64_t)row * ldo + c0, acc, valid, accumulate, vec_out);
}

// Number of work units (4 consecutive columns of one row, or one gate) of one problem.
__host__ __device__ inline int64_t bwd_finish_units(const BwdFinishArgs& a) {
  const int64_t c4r = (a.r + 3) >> 2, c4d = (a.d_in + 3) >> 2;
  const int64_t c8d = (a.d_in + 7) >> 3;   // diag(z) Q moves 8 columns (16 bytes) per unit
  return (a.dP ? (int64_t)a.d_out * c4r : 0) + (a.dQ ? (int64_t)a.r * c4d : 0) + (a.Qz ? (int64_t)a.r * c8d : 0) +
         (a.dlog_alpha ? (int64_t)a.r : 0);
}

template <typename TW>
__device__ __forceinline__ void bwd_finish_unit(const BwdFinishArgs& a, int64_t u) {
  const int c4r = (a.r + 3) >> 2, c4d = (a.d_in + 3) >> 2;
  const int64_t n_p = a.dP ? (int64_t)a.d_out * c4r : 0;
  const int64_t n_q = a.dQ ? (int64_t)a.r * c4d : 0;
  const int c8d = (a.d_in + 7) >> 3;
  const int64_t n_qz = a.Qz ? (int64_t)a.r * c8d : 0;
  constexpr int al = sizeof(TW) == 4 ? 15 : 7;   // 4 outputs: 16 B (fp32) or 8 B (bf16)
  if (u < n_p) {
    const bool vec_p = ((reinterpret_cast<uintptr_t>(a.dP) & al) == 0) && (a.lddp % 4 == 0);
    const int row = (int)(u / c4r), c0 = (int)(u % c4r) * 4;
    reduce_unit<TW>(a.slices_p, a.n_slices_p, a.slice_elems_p, a.ld_slice_p, row, c0, a.r, 1.f, (TW*)a.dP, a.lddp,
                    a.accumulate, vec_p);
  } else if (u < n_p + n_q) {
    const bool vec_q = ((reinterpret_cast<uintptr_t>(a.dQ) & al) == 0) && (a.lddq % 4 == 0);
    const int64_t v = u - n_p;
    const int row = (int)(v / c4d), c0 = (int)(v % c4d) * 4;
    reduce_unit<TW>(a.slices_q, a.n_slices_q, a.slice_elems_q, a.ld_slice_q, row, c0, a.d_in, a.z[row], (TW*)a.dQ, a.lddq,
                    a.accumulate, vec_q);
  } else if (u < n_p + n_q + n_qz) {
    const int v = (int)(u - n_p - n_q);
    const int row = v / c8d, c0 = (v - row * c8d) * 8;
    const int valid = min(8, a.d_in - c0);
    const float g = a.z[row];
    const __nv_bfloat16* q = a.Q + (int64_t)row * a.ldq + c0;
    __nv_bfloat16* o = a.Qz + (int64_t)row * a.ldqz + c0;
    if (valid == 8) {   // Q and Qz rows are 16-byte aligned (ld % 8 == 0)
      uint4 raw = *reinterpret_cast<const uint4*>(q);
      __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 x = __bfloat1622float2(h[i]);
        h[i] = __floats2bfloat162_rn(x.x * g, x.y * g);
      }
      *reinterpret_cast<uint4*>(o) = raw;
    } else {
      for (int i = 0; i < valid; ++i) o[i] = __float2bfloat16_rn(__bfloat162float(q[i]) * g);
    }
  } else {
    const int k = (int)(u - n_p - n_q - n_qz);
    float s = 0.f;
    for (int p = 0; p < a.n_part; ++p) s += a.dz_part[(int64_t)p * a.r + k];
    const float v = s * a.dz_dla[k];
    a.dlog_alpha[k] = a.accumulate ? a.dlog_alpha[k] + v : v;
  }
}

template <typename TW>
__global__ void __launch_bounds__(256)
bwd_finish_kernel(const BwdFinishArgs a) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t total = bwd_finish_units(a);
  for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (int64_t)gridDim.x * blockDim.x)
    bwd_finish_unit<TW>(a, u);
}

// The same for up to kFinishGroup matrices in one launch (grouped backward).
constexpr int kFinishGroup = 8;
struct BwdFinishGroup {
  BwdFinishArgs a[kFinishGroup];
  int64_t unit_begin[kFinishGroup + 1];
  int n;
};

template <typename TW>
__global__ void __launch_bounds__(256)
bwd_finish_group_kernel(const __grid_constant__ BwdFinishGroup g) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t total = g.unit_begin[g.n];
  for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (int64_t)gridDim.x * blockDim.x) {
    int i = 0;
#pragma unroll
    for (int j = 1; j < kFinishGroup; ++j)
      if (j < g.n && u >= g.unit_begin[j]) i = j;
    bwd_finish_unit<TW>(g.a[i], u - g.unit_begin[i]);
  }
}

// The second stage of dlog_alpha for many matrices in one launch: a training step may leave the partial row dots
// of every backward call in that call's workspace and add them up once, at the end of the step.  The number of
// partial vectors is read from the word the backward GEMM left next to them.  Partials are added in index order.
constexpr int kDlaGroup = 96;
struct DlaFinish { const float* dz_part; const int* n_part; int cap; const float* dz_dla; float* dla; int r; };
struct DlaFinishGroup { DlaFinish a[kDlaGroup]; int n; };

__global__ void __launch_bounds__(256)
dalpha_group_kernel(const __grid_constant__ DlaFinishGroup g, int accumulate) {
  pdl_wait();
  pdl_launch_dependents();
  const DlaFinish& a = g.a[blockIdx.y];
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= a.r) return;
  const int n_part = min(max(*a.n_part, 0), a.cap);
  float s = 0.f;
  for (int p = 0; p < n_part; ++p) s += a.dz_part[(int64_t)p * a.r + k];
  const float v = s * a.dz_dla[k];
  a.dla[k] = accumulate ? a.dla[k] + v : v;
}

// diag(z) Q of many matrices in one launch (it depends only on the gate sample and the weights, so a training
// step forms it once, right after sampling, for every matrix of the model).  16-byte units; rows are 16-byte aligned.
constexpr int kScaleGroup = 96;
struct ScaleRows { const __nv_bfloat16* Q; int64_t ldq; const float* z; __nv_bfloat16* Qz; int64_t ldqz; int rows, cols; };
struct ScaleRowsGroup {
  ScaleRows a[kScaleGroup];
  int n;
};

// blockIdx.y = matrix.  A block takes kScaleRows rows at a time, four per warp; a warp reads 512 consecutive bytes
// of each of its rows per pass and keeps the loads of its four rows (two passes) in flight before it stores.
constexpr int kScaleRows = 32;
__global__ void __launch_bounds__(256)
scale_rows_group_kernel(const __grid_constant__ ScaleRowsGroup g) {
  pdl_wait();
  pdl_launch_dependents();
  const ScaleRows& a = g.a[blockIdx.y];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r0 = blockIdx.x * kScaleRows; r0 < a.rows; r0 += gridDim.x * kScaleRows) {
    float gate[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = r0 + warp + 8 * i;
      gate[i] = row < a.rows ? __ldg(a.z + row) : 0.f;
    }
    for (int c0 = lane * 8; c0 < a.cols; c0 += 512) {
      uint4 raw[8];
      bool full[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int row = r0 + warp + 8 * (j & 3), c = c0 + 256 * (j >> 2);
        full[j] = row < a.rows && c + 8 <= a.cols;
        if (full[j]) raw[j] = __ldcs(reinterpret_cast<const uint4*>(a.Q + (int64_t)row * a.ldq + c));
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int row = r0 + warp + 8 * (j & 3), c = c0 + 256 * (j >> 2);
        if (full[j]) {
          __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw[j]);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 x = __bfloat1622float2(h[e]);
            h[e] = __floats2bfloat162_rn(x.x * gate[j & 3], x.y * gate[j & 3]);
          }
          *reinterpret_cast<uint4*>(a.Qz + (int64_t)row * a.ldqz + c) = raw[j];
        } else if (row < a.rows && c < a.cols) {            // ragged last piece of a row
          for (int k = 0; k < a.cols - c; ++k)
            a.Qz[(int64_t)row * a.ldqz + c + k] = __float2bfloat16_rn(__bfloat162float(a.Q[(int64_t)row * a.ldq + c + k]) * gate[j & 3]);
        }
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
fill_zero_2d_kernel(T* __restrict__ out, int64_t ld, int rows, int cols) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)rows * cols) return;
  out[(i / cols) * ld + (i % cols)] = from_f32<T>(0.f);
}

}  // namespace flop
