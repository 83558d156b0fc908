// Expected L0 size and augmented-Lagrangian penalty (Eq. 3 and Section 4.3).
//
// Three launches, no atomics, fixed summation order (bit-reproducible):
//   1. l0_chunk_kernel<false>: every block owns one chunk of kL0Chunk gates of ONE
//      segment and writes sum(pi_j) of the chunk (fp64) to scratch.
//   2. l0_finalize_kernel    : one block adds the chunk sums per segment in chunk
//      order, forms s, g, dg/dlambda and the gradient coefficient.
//   3. l0_chunk_kernel<true> : dlog_alpha_j += coef * size_seg * pi_j (1 - pi_j).
// Blocks find their (segment, chunk) from the segment table alone: chunk
// counts per segment are prefix-summed in shared memory by every block.
// The segment table lives in device memory, so the host cannot check it: the kernels
// do.  A table that needs more chunk sums than the scratch holds (`capacity`), or
// that points outside [0, n), touches nothing; the finalisation then reports
// FLOP_ERR_INVALID_ARG in the device status word and writes NaN to out4.
#pragma once
#include "common.cuh"

namespace flop {

constexpr int kL0Threads = 256;
constexpr int kL0PerThread = 32;                    // eight 16-byte vectors per thread
constexpr int kL0Chunk = kL0Threads * kL0PerThread;  // gates per block
constexpr int kL0MaxSeg = 4096;

struct L0Scratch {         // layout of the caller's workspace
  double coef;             // (lambda1 + 2 lambda2 (s - t)) / S
  double pad[31];
  double partial[1];       // [n_chunks_max]
};

// Fills seg_first_chunk[0..n_seg] (exclusive prefix of chunks per segment) in
// shared memory.  Serial per 16 segments per thread, then a block scan.
__device__ __forceinline__ void l0_chunk_table(const int64_t* __restrict__ seg_off, int n_seg, int* first_chunk,
                                               int* scan_scratch) {
  // thread t owns segments [t*per, (t+1)*per): per = 1 for up to 256 segments, so the table costs
  // one 16-byte read per thread instead of a fixed sixteen
  const int per = (n_seg + kL0Threads - 1) / kL0Threads;
  const int s0 = threadIdx.x * per;
  int sum = 0;
  for (int i = 0; i < per; ++i) {
    const int s = s0 + i;
    if (s < n_seg) {
      const int64_t len = seg_off[s + 1] - seg_off[s];
      sum += len > 0 ? (int)((len + kL0Chunk - 1) / kL0Chunk) : 0;
    }
  }
  int total;
  int base = block_exclusive_scan(sum, scan_scratch, &total);
  for (int i = 0; i < per; ++i) {
    const int s = s0 + i;
    if (s < n_seg) {
      first_chunk[s] = base;
      const int64_t len = seg_off[s + 1] - seg_off[s];
      base += len > 0 ? (int)((len + kL0Chunk - 1) / kL0Chunk) : 0;
    }
  }
  if (threadIdx.x == 0) first_chunk[n_seg] = total;
  __syncthreads();
}

// Largest s with first_chunk[s] <= b and a non-empty chunk range containing b.
__device__ __forceinline__ int l0_find_segment(const int* first_chunk, int n_seg, int b) {
  int lo = 0, hi = n_seg;  // invariant: first_chunk[lo] <= b < first_chunk[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (first_chunk[mid] <= b) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ float l0_pi(float a, float thr) { return __fdividef(1.0f, 1.0f + __expf(-(a - thr))); }

template <bool kGrad>
__global__ void __launch_bounds__(kL0Threads)
l0_chunk_kernel(const float* __restrict__ log_alpha, const int64_t* __restrict__ seg_off,
                const float* __restrict__ seg_size, int n_seg, float thr, L0Scratch* __restrict__ sc,
                float* __restrict__ dlog_alpha, int64_t n, int capacity) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int first_chunk[kL0MaxSeg + 1];
  __shared__ int scan_scratch[33];
  __shared__ double red[32];
  l0_chunk_table(seg_off, n_seg, first_chunk, scan_scratch);
  const int b = blockIdx.x;
  if (first_chunk[n_seg] > capacity) return;   // the table asks for more chunk sums than the scratch holds
  if (b >= first_chunk[n_seg]) {            // surplus block of the upper-bound grid
    return;
  }
  const int seg = l0_find_segment(first_chunk, n_seg, b);
  const int64_t lo = seg_off[seg] + (int64_t)(b - first_chunk[seg]) * kL0Chunk;
  const int64_t hi = min(seg_off[seg + 1], lo + (int64_t)kL0Chunk);
  if (lo < 0 || hi > n) return;             // a segment outside the gate vector: nothing is read or written
  // vector v of thread t covers gates lo + (v*256 + t)*4 .. +3: consecutive threads, consecutive 16 bytes
  constexpr int kVec = kL0PerThread / 4;
  const bool al_a = (reinterpret_cast<uintptr_t>(log_alpha + lo) & 15) == 0;
  double sum = 0.0;
  float w = 0.f;
  bool al_g = false;
  if (kGrad) {
    w = (float)(sc->coef * (double)seg_size[seg]);
    al_g = al_a && (reinterpret_cast<uintptr_t>(dlog_alpha + lo) & 15) == 0;
  }
#pragma unroll
  for (int v = 0; v < kVec; ++v) {
    const int64_t j0 = lo + ((int64_t)v * kL0Threads + threadIdx.x) * 4;
    if (j0 >= hi) continue;
    float a[4];
    const bool full = j0 + 4 <= hi;
    if (full && al_a) {
      const float4 t = __ldcs(reinterpret_cast<const float4*>(log_alpha + j0));
      a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = (j0 + i < hi) ? log_alpha[j0 + i] : 0.f;
    }
    if (!kGrad) {
      // the four probabilities of a vector are added in fp32 (each is in (0, 1): the group sum is exact to
      // 2^-22), the groups in fp64: a quarter of the fp64 conversions and additions, which bound this pass
      float p4[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) p4[i] = (j0 + i < hi) ? l0_pi(a[i], thr) : 0.f;
      sum += (double)((p4[0] + p4[1]) + (p4[2] + p4[3]));
    } else {
      float gsum[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // pi (1 - pi) = e / (1 + e)^2 with e = exp(-|alpha - thr|): no cancellation near pi = 1
        const float e = __expf(-fabsf(a[i] - thr));
        const float q = __fdividef(1.0f, 1.0f + e);
        gsum[i] = w * e * q * q;
      }
      if (full && al_g) {
        float4 g = *reinterpret_cast<float4*>(dlog_alpha + j0);
        g.x += gsum[0]; g.y += gsum[1]; g.z += gsum[2]; g.w += gsum[3];
        *reinterpret_cast<float4*>(dlog_alpha + j0) = g;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (j0 + i < hi) dlog_alpha[j0 + i] += gsum[i];
      }
    }
  }
  if (!kGrad) {
    sum = block_sum_f64(sum, red);
    if (threadIdx.x == 0) sc->partial[b] = sum;
  }
}

__global__ void __launch_bounds__(kL0Threads)
l0_finalize_kernel(const int64_t* __restrict__ seg_off, const float* __restrict__ seg_size, int n_seg,
                   const float* __restrict__ target, const float* __restrict__ lambda, L0Scratch* __restrict__ sc,
                   float* __restrict__ out4, float* __restrict__ seg_expected, int64_t n, int capacity) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int first_chunk[kL0MaxSeg + 1];
  __shared__ int scan_scratch[33];
  __shared__ double red_w[32], red_s[32];
  __shared__ int bad;
  if (threadIdx.x == 0) bad = 0;
  l0_chunk_table(seg_off, n_seg, first_chunk, scan_scratch);
  // the segments must partition [0, n): ascending offsets from 0 to n (the chunk sums of anything else were not written)
  for (int s = threadIdx.x; s < n_seg; s += blockDim.x)
    if (seg_off[s] < 0 || seg_off[s + 1] < seg_off[s] || seg_off[s + 1] > n) bad = 1;
  __syncthreads();
  if (first_chunk[n_seg] > capacity || bad || (n_seg > 0 && (seg_off[0] != 0 || seg_off[n_seg] != n))) {
    if (threadIdx.x == 0) {
      atomicExch(&g_device_status, (int)FLOP_ERR_INVALID_ARG);
      const float nan = __int_as_float(0x7fc00000);
      out4[0] = nan; out4[1] = nan; out4[2] = nan; out4[3] = nan;
      sc->coef = 0.0;
    }
    return;
  }
  // One warp per segment (segments w, w + nwarp, ...): lanes stride over the segment's chunk sums,
  // a butterfly adds them, and every warp keeps running totals over its own segments.  The
  // assignment is fixed, so the result is bit-reproducible.
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = kL0Threads / 32;
  double weighted = 0.0, total_size = 0.0;
  for (int s = warp; s < n_seg; s += nwarp) {
    double v = 0.0;
    for (int c = first_chunk[s] + lane; c < first_chunk[s + 1]; c += 32) v += sc->partial[c];
    v = warp_sum_f64(v);
    if (lane == 0 && seg_expected) seg_expected[s] = (float)v;
    const double size = (double)seg_size[s];
    weighted += size * v;
    total_size += size * (double)(seg_off[s + 1] - seg_off[s]);
  }
  if (lane == 0) { red_w[warp] = weighted; red_s[warp] = total_size; }
  __syncthreads();
  if (threadIdx.x == 0) {
    weighted = 0.0; total_size = 0.0;
    for (int w = 0; w < nwarp; ++w) { weighted += red_w[w]; total_size += red_s[w]; }
    const double s = total_size > 0.0 ? weighted / total_size : 0.0;
    const double diff = s - (double)target[0];
    const double l1 = (double)lambda[0], l2 = (double)lambda[1];
    out4[0] = (float)s;
    out4[1] = (float)(l1 * diff + l2 * diff * diff);
    out4[2] = (float)diff;
    out4[3] = (float)(diff * diff);
    sc->coef = total_size > 0.0 ? (l1 + 2.0 * l2 * diff) / total_size : 0.0;
  }
}

}  // namespace flop
