// Shared device helpers: status word, type conversion, block reductions/scans.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/flop.h"

namespace flop {

// Device status word: 0 = ok, otherwise a flop_status_t written by a kernel
// whose bounded wait gave up.  Read and cleared by flop_device_status().
__device__ int g_device_status = 0;

// Programmatic dependent launch: every kernel of the library is launched so that its prologue may
// overlap the tail of the kernel before it on the stream.  pdl_wait() blocks until all earlier
// kernels have completed and their writes are visible; it comes before the first access to
// global memory.  pdl_launch_dependents() lets the next kernel start its own prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void report_timeout() { atomicExch(&g_device_status, (int)FLOP_ERR_TIMEOUT); }

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block in a fixed order (butterfly inside each warp, then the
// warp totals added in warp order): the same inputs give the same bits.
// `scratch` holds at least 32 doubles.  Every thread gets the total.
__device__ __forceinline__ double block_sum_f64(double v, double* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
  v = warp_sum_f64(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < nwarp; ++w) t += scratch[w];
  return t;
}

// Exclusive prefix sum of one int per thread over the block, in thread order
// (ballot-free: shuffle scan inside the warp, warp totals in shared memory).
// `scratch` holds at least 33 ints.  Returns the exclusive prefix; *total gets
// the block total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* scratch, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) scratch[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < nwarp; ++w) {
    int s = scratch[w];
    if (w < warp) base += s;
    tot += s;
  }
  *total = tot;
  return base + inc - v;
}

}  // namespace flop
