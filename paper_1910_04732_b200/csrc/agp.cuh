// FLOP-AGP variant (Section 5 of the paper, baselines): magnitude-based pruning of the learnable
// diagonal mask G = diag(g) instead of hard-concrete gates, with an L1 term on the masks.
//
// One block per segment (weight matrix): the round(sparsity * r) entries of smallest |g| are pruned,
// the others keep their value.  The cut is found exactly by a 4-pass radix select on the bit
// pattern of |g| (monotone for non-negative floats); ties at the cut keep the lower indices, which
// a block scan over the tie flags decides.  z = g on kept entries, 0 elsewhere; dz/dg = [kept];
// seg_l1 = sum |g| of the segment (fp64 sum, fixed order); dg += l1 * sign(g) when requested.
// The forward/backward kernels are then used unchanged with z and dz/dg in place of the sampled
// gate and its derivative.
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kAgpThreads = 1024;

__global__ void __launch_bounds__(kAgpThreads)
agp_gates_kernel(const float* __restrict__ g, const int64_t* __restrict__ seg_off, const float* __restrict__ sparsity,
                 float l1, float* __restrict__ z, uint8_t* __restrict__ mask, float* __restrict__ dz_dg,
                 float* __restrict__ seg_l1, float* __restrict__ dg) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ double red[32];
  __shared__ int hist[256];
  __shared__ int scan_scratch[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  const int tid = threadIdx.x;
  const int64_t lo = seg_off[blockIdx.x];
  const int r = (int)(seg_off[blockIdx.x + 1] - lo);
  const float* gs = g + lo;
  // the count is decided in fp64, as the definition states it
  const int n_pruned = (int)floor((double)sparsity[0] * (double)r + 0.5);
  const int keep = max(0, min(r, r - n_pruned));
  double l1sum = 0.0;
  for (int j = tid; j < r; j += kAgpThreads) l1sum += (double)fabsf(gs[j]);
  l1sum = block_sum_f64(l1sum, red);
  if (tid == 0 && seg_l1) seg_l1[blockIdx.x] = (float)l1sum;
  uint32_t kth = 0;
  int need_eq = 0;
  if (keep > 0 && keep < r) {
    uint32_t prefix = 0, pmask = 0;
    int need = keep;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int j = tid; j < r; j += kAgpThreads) {
        const uint32_t key = __float_as_uint(fabsf(gs[j]));
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
  int base_eq = 0;
  for (int j0 = 0; j0 < r; j0 += kAgpThreads) {
    const int j = j0 + tid;
    float v = 0.f;
    int gt = 0, eq = 0;
    if (j < r) {
      v = gs[j];
      const uint32_t key = __float_as_uint(fabsf(v));
      if (keep >= r) gt = 1;
      else if (keep > 0) { gt = key > kth; eq = key == kth; }
    }
    int tot_eq = 0;
    const int rank_eq = base_eq + block_exclusive_scan(eq, scan_scratch, &tot_eq);
    base_eq += tot_eq;
    if (j < r) {
      const int kept = gt || (eq && rank_eq < need_eq);
      z[lo + j] = kept ? v : 0.f;
      if (mask) mask[lo + j] = (uint8_t)kept;
      if (dz_dg) dz_dg[lo + j] = kept ? 1.f : 0.f;
      if (dg) dg[lo + j] += l1 * (v > 0.f ? 1.f : (v < 0.f ? -1.f : 0.f));
    }
  }
}

}  // namespace flop
