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
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= r) return;
  float s = 0.f;
  for (int p = 0; p < n_part; ++p) s += dz_part[(int64_t)p * part_stride + k];
  const float v = s * dz_dla[k];
  dlog_alpha[k] = accumulate ? dlog_alpha[k] + v : v;
}

template <typename T>
__global__ void __launch_bounds__(256)
fill_zero_2d_kernel(T* __restrict__ out, int64_t ld, int rows, int cols) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)rows * cols) return;
  out[(i / cols) * ld + (i % cols)] = from_f32<T>(0.f);
}

}  // namespace flop
