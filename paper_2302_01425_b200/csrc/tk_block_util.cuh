// tk_block_util.cuh -- block-wide scan and sum used by the block-per-row kernels.
#pragma once

#include "tk_common.cuh"

namespace tk {

// Block-wide exclusive prefix over threads; total returned to all.  red: >= 33 slots.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* red, T* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  T inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  if (lane == 31) red[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    T w = (lane < nwarps) ? red[lane] : T(0);
    T winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      T up = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += up;
    }
    red[lane] = winc - w;                 // exclusive warp offsets
    if (lane == 31) red[32] = winc;       // grand total
  }
  __syncthreads();
  T res = red[warp] + inc - v;
  *total = red[32];
  __syncthreads();
  return res;
}

template <typename T>
__device__ __forceinline__ T block_sum(T v, T* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  T w = (lane < nwarps) ? red[lane] : T(0);
  w = warp_sum(w);
  __syncthreads();
  return w;
}

}  // namespace tk
