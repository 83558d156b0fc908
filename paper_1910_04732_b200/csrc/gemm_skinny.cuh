// Forward GEMM for 5..16 tokens, bf16 in, fp32 accumulate, bf16 out:
//     C[t, n] = col_scale[n] * sum_k A[t, k] B[n, k]          (A [T, K], B [N, K], both K-major)
//
// Between the weight-streaming CUDA-core kernel (T <= 4) and the 128-row tcgen05 tiles (which a
// batch this small fills to an eighth, at ~9 us of pipeline set-up per launch) the product is
// still bound by reading B once.  One warp owns eight output columns and walks K with warp-level
// m16n8k16 tensor-core instructions: the T rows of A (padded to a multiple of 16) sit in shared
// memory, every lane reads 16 contiguous bytes of one row of B per 32-wide K step, and the k
// positions inside a step are permuted identically for A and B so that those 16 bytes serve two
// instructions without a shuffle (a dot product does not care in which order k is visited).
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kSkinnyMaxT = 16;   // measured: 12-14 us up to 16 tokens, level with the tcgen05 path (20 us) at 32
constexpr int kSkinnyWarps = 8;
constexpr int kSkinnyPad = 32;   // elements added to a row of A in shared memory: rows land 16 banks apart

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int MT>   // row tiles of 16 tokens
__global__ void __launch_bounds__(32 * kSkinnyWarps)
skinny_gemm_kernel(const __nv_bfloat16* __restrict__ A, int64_t lda, const __nv_bfloat16* __restrict__ B, int64_t ldb,
                   __nv_bfloat16* __restrict__ C, int64_t ldc, const float* __restrict__ col_scale, int T, int N, int K,
                   int k_pad) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* As = reinterpret_cast<__nv_bfloat16*>(smem_raw);   // [16 MT][k_pad + kSkinnyPad], zero beyond T and K
  const int stride = k_pad + kSkinnyPad;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int e = tid * 8; e < 16 * MT * k_pad; e += blockDim.x * 8) {
    const int t = e / k_pad, k = e - t * k_pad;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (t < T) {
      if (k + 8 <= K) {
        v = *reinterpret_cast<const uint4*>(A + (int64_t)t * lda + k);      // rows are 16-byte aligned (ld % 8 == 0)
      } else {
        __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&v);
        for (int i = 0; i < 8 && k + i < K; ++i) h[i] = A[(int64_t)t * lda + k + i];
      }
    }
    *reinterpret_cast<uint4*>(As + (int64_t)t * stride + k) = v;
  }
  __syncthreads();
  const int g = lane >> 2, q = lane & 3;
  const int groups = (N + 7) >> 3;
  for (int ng = blockIdx.x * kSkinnyWarps + warp; ng < groups; ng += gridDim.x * kSkinnyWarps) {
    const int n = ng * 8 + g;                      // the row of B this lane reads
    const __nv_bfloat16* b = B + (int64_t)min(n, N - 1) * ldb;
    float acc[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[m][i] = 0.f;
    // Eight 32-wide K steps per trip: the eight 16-byte reads of B are issued together, so a warp has
    // 128 bytes per lane in flight instead of waiting for one read per step.
    for (int kk = 0; kk < K; kk += 256) {
      uint4 bvs[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int k = kk + 32 * u + 8 * q;
        bvs[u] = make_uint4(0, 0, 0, 0);
        if (n < N) {
          if (k + 8 <= K) {
            bvs[u] = __ldg(reinterpret_cast<const uint4*>(b + k));
          } else {
            __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&bvs[u]);
            for (int i = 0; i < 8 && k + i < K; ++i) h[i] = b[k + i];
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
      const int k0 = kk + 32 * u;
      if (k0 >= K) break;
      const int k = k0 + 8 * q;
      const uint4 bv = bvs[u];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        const uint4 lo = *reinterpret_cast<const uint4*>(As + (int64_t)(m * 16 + g) * stride + k);
        const uint4 hi = *reinterpret_cast<const uint4*>(As + (int64_t)(m * 16 + g + 8) * stride + k);
        mma_bf16_16816(acc[m], lo.x, hi.x, lo.y, hi.y, bv.x, bv.y);
        mma_bf16_16816(acc[m], lo.z, hi.z, lo.w, hi.w, bv.z, bv.w);
      }
      }
    }
    const int nc = ng * 8 + 2 * q;                 // the two columns this lane holds
    const float s0 = (col_scale && nc < N) ? __ldg(col_scale + nc) : 1.f;
    const float s1 = (col_scale && nc + 1 < N) ? __ldg(col_scale + nc + 1) : 1.f;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int t = m * 16 + g + 8 * h;
        if (t < T) {
          if (nc < N) C[(int64_t)t * ldc + nc] = __float2bfloat16_rn(acc[m][2 * h] * s0);
          if (nc + 1 < N) C[(int64_t)t * ldc + nc + 1] = __float2bfloat16_rn(acc[m][2 * h + 1] * s1);
        }
      }
    }
  }
}

}  // namespace flop
