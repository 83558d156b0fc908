// Hard-concrete gate sampler (Section 3 of the paper) driven by Philox4x32-10.
//
// One thread draws one Philox block = four gates, so loads and stores are
// 16-byte vectors.  The arithmetic runs in fp32; the two clamp decisions
// (z > 0, z < 1) are taken in logit space, t = logit(u) + alpha against
// c0 = beta log(-gamma/zeta) and c1 = beta log((1-gamma)/(zeta-1)), and any
// gate whose t lies within kBand of c0 or c1 is re-evaluated in fp64 with the
// formulas in the paper's order, so the mask equals the fp64 evaluation.
#pragma once
#include "common.cuh"

namespace flop {

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
  // Philox-4x32, ten rounds (Salmon et al., SC'11): two 32x32->64 multiplies
  // per round, xor with the key and the neighbouring words, Weyl key schedule.
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(M0, c.x), lo0 = M0 * c.x;
    const uint32_t hi1 = __umulhi(M1, c.z), lo1 = M1 * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += W0;
    k.y += W1;
  }
  return c;
}

struct GateConsts {
  float inv_beta, gamma, zeta, c0, c1;   // fp32 fast path
  double beta_d, gamma_d, zeta_d;        // exact images of the fp32 parameters
};

constexpr float kBand = 2.5e-5f;  // |t - c| below this -> fp64; fp32 error of t is < 5.3e-6 (see gate_one)

__device__ __forceinline__ void gate_fp64(float alpha, float u, const GateConsts& g, float& z, int& m, float& d) {
  // The sampler exactly as printed, one rounded operation at a time.
  const double ud = (double)u;
  const double t = __ddiv_rn(__dadd_rn(__dsub_rn(log(ud), log(__dsub_rn(1.0, ud))), (double)alpha), g.beta_d);
  const double s = __ddiv_rn(1.0, __dadd_rn(1.0, exp(-t)));
  const double range = __dsub_rn(g.zeta_d, g.gamma_d);
  const double sb = __dadd_rn(__dmul_rn(s, range), g.gamma_d);
  const double zc = fmin(1.0, fmax(0.0, sb));
  m = zc > 0.0;
  z = (float)zc;
  d = (sb > 0.0 && sb < 1.0) ? (float)(range * s * (1.0 - s) / g.beta_d) : 0.f;
}

__device__ __forceinline__ void gate_one(float alpha, uint32_t bits, const GateConsts& g, float& z, int& m, float& d) {
  const float u = ((float)(bits >> 9) + 0.5f) * 1.1920928955078125e-7f;  // 2^-23; exact
  // logit(u) with the fast intrinsics: u / (1 - u) is within 2 ulp, __logf within 2 ulp of a value of
  // magnitude <= 16.7 (4e-6), the sum with alpha rounds once more (1e-6): t is off by < 5.3e-6, a fifth
  // of the band that sends a gate to fp64
  const float t = __logf(__fdividef(u, 1.0f - u)) + alpha;
  if (fabsf(t - g.c0) < kBand || fabsf(t - g.c1) < kBand || !(fabsf(t) < 1e30f)) {
    gate_fp64(alpha, u, g, z, m, d);
  } else if (t < g.c0) {
    z = 0.f; m = 0; d = 0.f;
  } else if (t > g.c1) {
    z = 1.f; m = 1; d = 0.f;
  } else {
    const float s = __fdividef(1.0f, 1.0f + __expf(-t * g.inv_beta));   // |t / beta| < 2.5 here: a few ulp
    const float range = g.zeta - g.gamma;
    z = fminf(1.0f, fmaxf(s * range + g.gamma, 1e-30f));
    m = 1;
    d = range * s * (1.0f - s) * g.inv_beta;
  }
}

__global__ void __launch_bounds__(256)
gate_sample_kernel(const float* __restrict__ log_alpha, int64_t n, GateConsts g, uint2 key, uint64_t offset_host,
                   const uint64_t* __restrict__ offset_dev,
                   float* __restrict__ z, uint8_t* __restrict__ mask, float* __restrict__ dz_dla, int vec_ok) {
  pdl_wait();
  pdl_launch_dependents();
  // the counter offset may also live in device memory, so that a captured launch can advance it
  const uint64_t offset = offset_host + (offset_dev ? *offset_dev : 0ull);
  const int64_t nblk = (n + 3) >> 2;
#pragma unroll 2
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblk; b += (int64_t)gridDim.x * blockDim.x) {
    const uint64_t ctr = offset + (uint64_t)b;
    const uint4 x = philox4x32_10(make_uint4((uint32_t)ctr, (uint32_t)(ctr >> 32), 0u, 0u), key);
    const uint32_t bits[4] = {x.x, x.y, x.z, x.w};
    const int64_t j0 = b << 2;
    float zz[4], dd[4];
    int mm[4];
    if (vec_ok && j0 + 4 <= n) {
      const float4 a = __ldcs(reinterpret_cast<const float4*>(log_alpha + j0));   // streamed once: do not keep in cache
      const float aa[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) gate_one(aa[i], bits[i], g, zz[i], mm[i], dd[i]);
      __stcs(reinterpret_cast<float4*>(z + j0), make_float4(zz[0], zz[1], zz[2], zz[3]));
      if (mask) __stcs(reinterpret_cast<uchar4*>(mask + j0), make_uchar4(mm[0], mm[1], mm[2], mm[3]));
      if (dz_dla) __stcs(reinterpret_cast<float4*>(dz_dla + j0), make_float4(dd[0], dd[1], dd[2], dd[3]));
    } else {
      for (int i = 0; i < 4 && j0 + i < n; ++i) {
        gate_one(log_alpha[j0 + i], bits[i], g, zz[i], mm[i], dd[i]);
        z[j0 + i] = zz[i];
        if (mask) mask[j0 + i] = (uint8_t)mm[i];
        if (dz_dla) dz_dla[j0 + i] = dd[i];
      }
    }
  }
}

}  // namespace flop
