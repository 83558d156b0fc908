// Forward GEMM for a handful of tokens (T <= 4), bf16 in, fp32 accumulate, bf16 out:
//     C[t, n] = col_scale[n] * sum_k A[t, k] B[n, k]          (A [T, K], B [N, K], both K-major)
//
// At T = 1..4 (pruned inference, batch x sequence of a few tokens) the product is a
// weight-streaming problem: every row of B is read once and used T times, a 128-row tensor-core
// tile would be at most a quarter full, and a tensor-core launch costs ~9 us of pipeline set-up
// against ~1 us of weight traffic.  Here one warp owns one output column n: its lanes stride over
// K with 16-byte loads of B[n, :], multiply with the T rows of A held in shared memory, and a
// shuffle tree adds the 32 partial sums per token.  Bound: HBM/L2 read of B.  Measured on the
// 1024 -> 4096, k = 412 inference case: 6.3 / 8.3 / 10.3 / 14.4 us at T = 1 / 2 / 4 / 8; from T = 5 the
// warp-level tensor-core kernel (gemm_skinny.cuh, 12 us) is faster.
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kSmallTMax = 4;
constexpr int kSmallTWarps = 8;

template <int TT>   // TT = tokens rounded up to 1, 2 or 4 (accumulators per lane)
__global__ void __launch_bounds__(32 * kSmallTWarps)
small_t_gemm_kernel(const __nv_bfloat16* __restrict__ A, int64_t lda, const __nv_bfloat16* __restrict__ B, int64_t ldb,
                    __nv_bfloat16* __restrict__ C, int64_t ldc, const float* __restrict__ col_scale, int T, int N, int K,
                    int k_pad) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* As = reinterpret_cast<__nv_bfloat16*>(smem_raw);   // [TT][k_pad], zero beyond T and K
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int e = tid * 8; e < TT * k_pad; e += blockDim.x * 8) {
    const int t = e / k_pad, k = e - t * k_pad;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (t < T) {
      if (k + 8 <= K) {
        v = *reinterpret_cast<const uint4*>(A + (int64_t)t * lda + k);    // rows are 16-byte aligned (ld % 8 == 0)
      } else {
        __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&v);
        for (int i = 0; i < 8 && k + i < K; ++i) h[i] = A[(int64_t)t * lda + k + i];
      }
    }
    *reinterpret_cast<uint4*>(As + e) = v;
  }
  __syncthreads();
  for (int n = blockIdx.x * kSmallTWarps + warp; n < N; n += gridDim.x * kSmallTWarps) {
    const __nv_bfloat16* b = B + (int64_t)n * ldb;
    float acc[TT];
#pragma unroll
    for (int t = 0; t < TT; ++t) acc[t] = 0.f;
    for (int k = lane * 8; k < K; k += 32 * 8) {
      uint4 bv = make_uint4(0, 0, 0, 0);
      if (k + 8 <= K) {
        bv = __ldg(reinterpret_cast<const uint4*>(b + k));
      } else {
        __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&bv);
        for (int i = 0; i < 8 && k + i < K; ++i) h[i] = b[k + i];
      }
      const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&bv);
      float2 bf[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) bf[i] = __bfloat1622float2(bh[i]);
#pragma unroll
      for (int t = 0; t < TT; ++t) {
        const uint4 av = *reinterpret_cast<const uint4*>(As + t * k_pad + k);
        const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&av);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 af = __bfloat1622float2(ah[i]);
          acc[t] = fmaf(af.x, bf[i].x, acc[t]);
          acc[t] = fmaf(af.y, bf[i].y, acc[t]);
        }
      }
    }
    const float sc = col_scale ? __ldg(col_scale + n) : 1.f;
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      float v = acc[t];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && t < T) C[(int64_t)t * ldc + n] = __float2bfloat16_rn(v * sc);
    }
  }
}

}  // namespace flop
