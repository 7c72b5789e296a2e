// tk_team.cuh -- a row shared by a team of lanes: G lanes of one warp (32 / G rows per warp) or
// W whole warps.  The only exchange between the lanes of a row is a sum: shuffles inside the warp,
// then, for W > 1, one shared-memory slot per warp and a named barrier over the team's warps.
#pragma once

#include "tk_common.cuh"

namespace tk {

constexpr int kTeamWarps = 4;               // warps per thread block when a row needs at most that many

// threads per block of a kernel whose rows take W warps
constexpr int team_threads(int W) { return W > kTeamWarps ? W * 32 : kTeamWarps * 32; }
// blocks per SM for which the register budget is set, given the warps per SM wanted
constexpr int team_min_blocks(int warps_per_sm, int W) {
  const int b = warps_per_sm * 32 / team_threads(W);
  return b < 1 ? 1 : b;
}

template <int G>
__device__ __forceinline__ float team_gsum(float v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int G>
__device__ __forceinline__ int team_gsum(int v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int G>
__device__ __forceinline__ float team_gmin(float v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ void team_barrier(int bar, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(threads) : "memory");
}

// Sum of NV (<= 3) values and of one packed pair of counts over the lanes of a row.  red: the team's
// W * 4 words for this phase; the caller alternates between two such buffers, so one barrier per sum
// is enough (a warp can be at most one sum ahead of the slowest warp of its team).  Every warp adds
// the slots in the same order: all lanes of the team end up with identical results.
template <int G, int W, int NV>
__device__ __forceinline__ void team_allsum(float (&v)[NV], uint32_t& packed, float* red, int wit, int lane, int bar) {
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = team_gsum<G>(v[i]);
  packed = (uint32_t)team_gsum<G>((int)packed);
  if (W > 1) {
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < NV; ++i) red[wit * 4 + i] = v[i];
      red[wit * 4 + 3] = __uint_as_float(packed);
    }
    team_barrier(bar, W * 32);
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = 0.0f;
    packed = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] += red[w * 4 + i];
      packed += __float_as_uint(red[w * 4 + 3]);
    }
  }
}

}  // namespace tk
