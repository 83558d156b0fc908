// Gated adaptive embedding of one word cluster (Section 4.2 of the paper): E~ = E G O.
// The lookup replaces the first GEMM of the gated layer by a row gather; the projection with O
// and the backward products are the tensor-core GEMMs used everywhere else.
//   embed_gather_kernel : H'[t, :] = E[ids[t], :] * z                       (one warp per token)
//   embed_bwd_kernel    : dE[ids[t], :] += dH'[t, :] * z   (fp32 atomic adds: rows repeat across tokens)
//                         part[b][k]    = sum over the block's tokens of E[ids[t], k] dH'[t, k]
//                         (the per-block partial sums of dz are then added in block order)
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kEmbWarps = 8;
constexpr int kEmbTokensPerWarp = 8;   // tokens a warp walks in the backward kernel

__global__ void __launch_bounds__(32 * kEmbWarps)
embed_gather_kernel(const int32_t* __restrict__ ids, int T, const __nv_bfloat16* __restrict__ E, int64_t lde, int n_rows,
                    const float* __restrict__ z, int d_i, __nv_bfloat16* __restrict__ H, int64_t ldh) {
  pdl_wait();
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * kEmbWarps + warp;
  if (t >= T) return;
  const int w = min(max(ids[t], 0), n_rows - 1);      // out-of-range ids are clamped, never dereferenced
  const __nv_bfloat16* e = E + (int64_t)w * lde;
  __nv_bfloat16* h = H + (int64_t)t * ldh;
  for (int k = lane * 8; k < d_i; k += 32 * 8) {
    if (k + 8 <= d_i) {
      uint4 raw = *reinterpret_cast<const uint4*>(e + k);
      __nv_bfloat16* v = reinterpret_cast<__nv_bfloat16*>(&raw);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __float2bfloat16_rn(__bfloat162float(v[i]) * __ldg(z + k + i));
      *reinterpret_cast<uint4*>(h + k) = raw;
    } else {
      for (int i = k; i < d_i; ++i) h[i] = __float2bfloat16_rn(__bfloat162float(e[i]) * z[i]);
    }
  }
}

// Block b handles tokens [b * 64, b * 64 + 64): warp w its 8 consecutive tokens.  A lane owns 8
// consecutive columns of every 256-column chunk (16-byte loads of dH' and E), so the per-column
// partial sums of dz need no cross-lane step; the eight warps' partials are added in warp order
// through shared memory.  dE takes 16-byte vector atomic adds when its rows allow them.
__global__ void __launch_bounds__(32 * kEmbWarps)
embed_bwd_kernel(const int32_t* __restrict__ ids, int T, const __nv_bfloat16* __restrict__ E, int64_t lde, int n_rows,
                 const float* __restrict__ z, int d_i, const __nv_bfloat16* __restrict__ dH, int64_t lddh,
                 float* __restrict__ dE, int64_t ldde, float* __restrict__ part) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ float red[];   // [kEmbWarps][d_i]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = (blockIdx.x * kEmbWarps + warp) * kEmbTokensPerWarp;
  const bool vec_de = dE && (reinterpret_cast<uintptr_t>(dE) & 15) == 0 && (ldde % 4) == 0;
  for (int k = lane * 8; k < d_i; k += 32 * 8) {
    const int nk = min(8, d_i - k);
    float zk[8], acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { zk[i] = i < nk ? z[k + i] : 0.f; acc[i] = 0.f; }
    for (int i = 0; i < kEmbTokensPerWarp; ++i) {
      const int t = t0 + i;
      if (t >= T) break;
      const int w = min(max(ids[t], 0), n_rows - 1);
      float gv[8], ev[8];
      if (nk == 8) {   // rows of dH' and E are 16-byte aligned (ld % 8 == 0)
        const uint4 graw = *reinterpret_cast<const uint4*>(dH + (int64_t)t * lddh + k);
        const uint4 eraw = *reinterpret_cast<const uint4*>(E + (int64_t)w * lde + k);
        const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&graw);
        const __nv_bfloat162* eh = reinterpret_cast<const __nv_bfloat162*>(&eraw);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 a = __bfloat1622float2(gh[j]), c = __bfloat1622float2(eh[j]);
          gv[2 * j] = a.x; gv[2 * j + 1] = a.y; ev[2 * j] = c.x; ev[2 * j + 1] = c.y;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          gv[j] = j < nk ? __bfloat162float(dH[(int64_t)t * lddh + k + j]) : 0.f;
          ev[j] = j < nk ? __bfloat162float(E[(int64_t)w * lde + k + j]) : 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = fmaf(ev[j], gv[j], acc[j]);
      if (dE) {
        float* o = dE + (int64_t)w * ldde + k;
        if (vec_de && nk == 8) {
          atomicAdd(reinterpret_cast<float4*>(o), make_float4(gv[0] * zk[0], gv[1] * zk[1], gv[2] * zk[2], gv[3] * zk[3]));
          atomicAdd(reinterpret_cast<float4*>(o + 4), make_float4(gv[4] * zk[4], gv[5] * zk[5], gv[6] * zk[6], gv[7] * zk[7]));
        } else {
          for (int j = 0; j < nk; ++j)
            if (zk[j] != 0.f) atomicAdd(o + j, gv[j] * zk[j]);
        }
      }
    }
    for (int j = 0; j < nk; ++j) red[warp * d_i + k + j] = acc[j];
  }
  __syncthreads();
  if (part) {
    for (int k = threadIdx.x; k < d_i; k += blockDim.x) {
      float s = 0.f;
      for (int w = 0; w < kEmbWarps; ++w) s += red[w * d_i + k];
      part[(int64_t)blockIdx.x * d_i + k] = s;
    }
  }
}

}  // namespace flop
