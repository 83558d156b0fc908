// Hard-concrete gate sampler (Section 3 of the paper) driven by Philox4x32-10.
//
// One thread draws one Philox block = four gates, so loads and stores are
// 16-byte vectors.  The arithmetic runs in fp32; the two clamp decisions
// (z > 0, z < 1) are taken in logit space, t = logit(u) + alpha against
// c0 = beta log(-gamma/zeta) and c1 = beta log((1-gamma)/(zeta-1)), and any
// gate whose t lies within kBand of c0 or c1 is re-evaluated in fp64 (together with
// the other three gates of its thread) with the formulas in the paper's order, so the
// mask equals the fp64 evaluation.
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
  float inv_beta, neg_inv_beta_log2e, gamma, zeta, c0, c1;   // fp32 fast path
  double beta_d, gamma_d, zeta_d;        // exact images of the fp32 parameters
};

constexpr float kBand = 2.5e-5f;  // |t - c| below this -> fp64; fp32 error of t is < 5.3e-6 (see gate_one)

// The sampler exactly as printed, one rounded fp64 operation at a time.
__device__ __forceinline__ void gate_fp64(float alpha, float u, const GateConsts& g, float& z, int& m, float& d) {
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

// Four gates in fp64, stored straight to memory.  Out of line and all by value: it runs for about one
// thread in 10^4, and this way it costs the fast path neither registers nor instruction-cache space.
__device__ __noinline__ void gate_fp64_store4(float4 a, float4 u, GateConsts g, float* z, uint8_t* mask, float* dz_dla) {
  const float aa[4] = {a.x, a.y, a.z, a.w}, uu[4] = {u.x, u.y, u.z, u.w};
  float zz[4], dd[4];
  int mm[4];
#pragma unroll 1
  for (int i = 0; i < 4; ++i) gate_fp64(aa[i], uu[i], g, zz[i], mm[i], dd[i]);
  *reinterpret_cast<float4*>(z) = make_float4(zz[0], zz[1], zz[2], zz[3]);
  if (mask) *reinterpret_cast<uchar4*>(mask) = make_uchar4(mm[0], mm[1], mm[2], mm[3]);
  if (dz_dla) *reinterpret_cast<float4*>(dz_dla) = make_float4(dd[0], dd[1], dd[2], dd[3]);
}

// Special-function approximations with denormals flushed to zero (no argument of the fast path is ever
// denormal: u / (1 - u) >= 2^-24, exp arguments are clamped to +-2.5), which spares the range fix-up code
// the compiler otherwise wraps around every one of them.
__device__ __forceinline__ float lg2_ftz(float x) { float y; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float ex2_ftz(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rcp_ftz(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// fp32 fast path of one gate.  Returns true when t lies within kBand of a clamp threshold (or is not
// finite): the caller then re-evaluates that gate with gate_fp64.  The rare branch is kept out of this
// function so that the four gates of a thread compile to one straight run of arithmetic.
__device__ __forceinline__ bool gate_one(float alpha, uint32_t bits, const GateConsts& g, float& u, float& z, int& m, float& d) {
  // u = ((bits >> 9) + 1/2) 2^-23, formed without an integer-to-float conversion (which shares the
  // special-function unit with log and exp): the 23 bits become the mantissa of a float in [1, 2), and
  // subtracting 1 - 2^-24 leaves (2k + 1) 2^-24 exactly.
  u = __uint_as_float(0x3F800000u | (bits >> 9)) - 0.999999940395355224609375f;
  // logit(u) with the approximate units: u / (1 - u) is within 2 ulp, the logarithm within 2 ulp of a value
  // of magnitude <= 16.7 (4e-6), the sum with alpha rounds once more (1e-6): t is off by < 5.3e-6, a fifth
  // of the band that sends a gate to fp64
  const float t = fmaf(lg2_ftz(u * rcp_ftz(1.0f - u)), 0.693147182464599609375f, alpha);
  const float tc = fminf(fmaxf(t, g.c0), g.c1);                               // keeps exp() in range: |tc / beta| < 2.5
  const float s = rcp_ftz(1.0f + ex2_ftz(tc * g.neg_inv_beta_log2e));         // a few ulp
  const float range = g.zeta - g.gamma;
  const bool below = t < g.c0, above = t > g.c1;
  z = below ? 0.f : (above ? 1.f : fminf(1.0f, fmaxf(s * range + g.gamma, 1e-30f)));
  m = below ? 0 : 1;
  d = (below || above) ? 0.f : range * s * (1.0f - s) * g.inv_beta;
  return fabsf(t - g.c0) < kBand || fabsf(t - g.c1) < kBand || !(fabsf(t) < 1e30f);
}

// 8 blocks of 256 threads per SM (32 registers a thread): with every warp slot filled the special-function and
// integer work of one warp hides behind the memory traffic of the others (measured 172 us against 185 us at
// 5 blocks per SM for 2^26 gates).
__global__ void __launch_bounds__(256, 8)
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
      float uu[4];
      bool redo = false;
#pragma unroll
      for (int i = 0; i < 4; ++i) redo |= gate_one(aa[i], bits[i], g, uu[i], zz[i], mm[i], dd[i]);
      if (redo) {   // about one thread in 10^4: all four gates again in fp64
        gate_fp64_store4(a, make_float4(uu[0], uu[1], uu[2], uu[3]), g, z + j0, mask ? mask + j0 : nullptr, dz_dla ? dz_dla + j0 : nullptr);
        continue;
      }
      __stcs(reinterpret_cast<float4*>(z + j0), make_float4(zz[0], zz[1], zz[2], zz[3]));
      if (mask) __stcs(reinterpret_cast<uchar4*>(mask + j0), make_uchar4(mm[0], mm[1], mm[2], mm[3]));
      if (dz_dla) __stcs(reinterpret_cast<float4*>(dz_dla + j0), make_float4(dd[0], dd[1], dd[2], dd[3]));
    } else {
      for (int i = 0; i < 4 && j0 + i < n; ++i) {
        float u;
        const float a = log_alpha[j0 + i];
        if (gate_one(a, bits[i], g, u, zz[i], mm[i], dd[i])) gate_fp64(a, u, g, zz[i], mm[i], dd[i]);
        z[j0 + i] = zz[i];
        if (mask) mask[j0 + i] = (uint8_t)mm[i];
        if (dz_dla) dz_dla[j0 + i] = dd[i];
      }
    }
  }
}

}  // namespace flop
