// fp32 FMA GEMM for the FLOP_F32 storage type: C[M,N] = sum_k A(m,k) B(n,k).
//
// The tensor cores have no true fp32 mode, and the fp32 configuration is held
// to 1e-5 relative error, so this path multiplies and accumulates in fp32 on
// the CUDA cores.  Operands are addressed by strides, which covers all six
// GEMMs of the layer (forward, and the backward ones that contract over
// tokens or over d_out) without transposes.  64x64x16 tiles, 4x4 per thread.
#pragma once
#include "common.cuh"

namespace flop {

struct SimtGemmArgs {
  const float* A; int64_t a_sm, a_sk;   // A(m,k) = A[m*a_sm + k*a_sk]
  const float* B; int64_t b_sn, b_sk;   // B(n,k) = B[n*b_sn + k*b_sk]
  float* C; int64_t ldc;                // C[m*ldc + n]
  int M, N, K;
  const float* col_scale;               // nullable: C[m,n] *= col_scale[n]
  const float* row_scale;               // nullable: C[m,n] *= row_scale[m]
  int accumulate;                       // C += instead of C =
};

__global__ void __launch_bounds__(256)
simt_gemm_kernel(SimtGemmArgs p) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tm = (tid >> 4) * 4, tn = (tid & 15) * 4;
  float acc[4][4] = {};
  const bool a_kfast = p.a_sk == 1, b_kfast = p.b_sk == 1;
  for (int k0 = 0; k0 < p.K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = tid + i * 256;   // 0..1023
      int m, k;
      if (a_kfast) { m = e >> 4; k = e & 15; } else { k = e >> 6; m = e & 63; }
      const int gm = m0 + m, gk = k0 + k;
      As[k][m] = (gm < p.M && gk < p.K) ? p.A[(int64_t)gm * p.a_sm + (int64_t)gk * p.a_sk] : 0.f;
      int n, kb;
      if (b_kfast) { n = e >> 4; kb = e & 15; } else { kb = e >> 6; n = e & 63; }
      const int gn = n0 + n, gkb = k0 + kb;
      Bs[kb][n] = (gn < p.N && gkb < p.K) ? p.B[(int64_t)gn * p.b_sn + (int64_t)gkb * p.b_sk] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][tm]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tn]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + tm + i;
    if (gm >= p.M) continue;
    const float rs = p.row_scale ? p.row_scale[gm] : 1.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tn + j;
      if (gn >= p.N) continue;
      float v = acc[i][j] * rs;
      if (p.col_scale) v *= p.col_scale[gn];
      float* c = p.C + (int64_t)gm * p.ldc + gn;
      *c = p.accumulate ? *c + v : v;
    }
  }
}

}  // namespace flop
