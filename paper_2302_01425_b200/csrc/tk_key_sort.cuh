// tk_key_sort.cuh -- sorting network on 32-bit float KEYS held by G lanes of a warp, E = 8 or 16
// keys per lane: the 19-comparator 8-sorter per lane, bitonic merges inside the lane and across
// lanes through shuffles.  A compare-exchange is one max and one min.  After group_sort_keys lane
// `lig` holds sorted ranks [E lig, E lig + E), descending.
#pragma once

#include "tk_common.cuh"

namespace tk {

__device__ __forceinline__ void cef(float& a, float& b) {   // a >= b after
  const float hi = fmaxf(a, b), lo = fminf(a, b);
  a = hi; b = lo;
}
__device__ __forceinline__ void sort8f(float (&r)[8]) {       // the 19-comparator network, descending
  cef(r[0], r[1]); cef(r[2], r[3]); cef(r[4], r[5]); cef(r[6], r[7]);
  cef(r[0], r[2]); cef(r[1], r[3]); cef(r[4], r[6]); cef(r[5], r[7]);
  cef(r[1], r[2]); cef(r[5], r[6]); cef(r[0], r[4]); cef(r[3], r[7]);
  cef(r[1], r[5]); cef(r[2], r[6]);
  cef(r[1], r[4]); cef(r[3], r[6]);
  cef(r[2], r[4]); cef(r[3], r[5]);
  cef(r[3], r[4]);
}
__device__ __forceinline__ void merge8f(float (&r)[8]) {      // bitonic -> descending
  cef(r[0], r[4]); cef(r[1], r[5]); cef(r[2], r[6]); cef(r[3], r[7]);
  cef(r[0], r[2]); cef(r[1], r[3]); cef(r[4], r[6]); cef(r[5], r[7]);
  cef(r[0], r[1]); cef(r[2], r[3]); cef(r[4], r[5]); cef(r[6], r[7]);
}
template <int E>
__device__ __forceinline__ void lane_sort_f(float (&r)[E]);
template <>
__device__ __forceinline__ void lane_sort_f<8>(float (&r)[8]) { sort8f(r); }
template <int E>
__device__ __forceinline__ void lane_merge_f(float (&r)[E]) {   // bitonic -> descending
#pragma unroll
  for (int stride = E >> 1; stride > 0; stride >>= 1) {
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const int j = i ^ stride;
      if (j > i) cef(r[i], r[j]);
    }
  }
}
template <>
__device__ __forceinline__ void lane_sort_f<16>(float (&r)[16]) {
  float hi[8], lo[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { hi[i] = r[i]; lo[i] = r[i + 8]; }
  sort8f(hi); sort8f(lo);
#pragma unroll
  for (int i = 0; i < 8; ++i) cef(hi[i], lo[7 - i]);      // element against its mirror: two bitonic halves
  merge8f(hi); merge8f(lo);
#pragma unroll
  for (int i = 0; i < 8; ++i) { r[i] = hi[i]; r[i + 8] = lo[i]; }
}

template <>
__device__ __forceinline__ void lane_sort_f<32>(float (&r)[32]) {
  float hi[16], lo[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) { hi[i] = r[i]; lo[i] = r[i + 16]; }
  lane_sort_f<16>(hi); lane_sort_f<16>(lo);
#pragma unroll
  for (int i = 0; i < 16; ++i) cef(hi[i], lo[15 - i]);     // element against its mirror: two bitonic halves
  lane_merge_f<16>(hi); lane_merge_f<16>(lo);
#pragma unroll
  for (int i = 0; i < 16; ++i) { r[i] = hi[i]; r[i + 16] = lo[i]; }
}

template <int G, int E>
__device__ __forceinline__ void group_sort_keys(float (&r)[E], int lig, unsigned mask) {
  lane_sort_f<E>(r);
  // 16 or 32 keys per lane: the rounds and lane stages are loops (a round is a few hundred
  // instructions; unrolled, the network is thousands that every warp fetches once per row).
  // Measured per 2^25 elements: n = 512 324 -> 313 us (p = 4/3: 392 -> 365), n = 1024 422 -> 411;
  // with 8 keys per lane the loops lose (n = 128: 175 -> 203 us), so those stay unrolled.
#pragma unroll (E >= 16 ? 1 : 5)
  for (int size = 2; size <= G; size <<= 1) {
    {
      const bool keepmax = (lig & (size >> 1)) == 0;
      if (E <= 16) {
        float o[E];
#pragma unroll
        for (int i = 0; i < E; ++i) o[i] = __shfl_xor_sync(mask, r[E - 1 - i], size - 1);
#pragma unroll
        for (int i = 0; i < E; ++i) r[i] = keepmax ? fmaxf(r[i], o[i]) : fminf(r[i], o[i]);
      } else {                                    // fewer live registers: slot i and its mirror together
#pragma unroll
        for (int i = 0; i < E / 2; ++i) {
          const float oa = __shfl_xor_sync(mask, r[E - 1 - i], size - 1);
          const float ob = __shfl_xor_sync(mask, r[i], size - 1);
          r[i] = keepmax ? fmaxf(r[i], oa) : fminf(r[i], oa);
          r[E - 1 - i] = keepmax ? fmaxf(r[E - 1 - i], ob) : fminf(r[E - 1 - i], ob);
        }
      }
    }
#pragma unroll (E >= 16 ? 1 : 5)
    for (int st = size >> 2; st >= 1; st >>= 1) {
      const bool keepmax = (lig & st) == 0;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float o = __shfl_xor_sync(mask, r[i], st);
        r[i] = keepmax ? fmaxf(r[i], o) : fminf(r[i], o);
      }
    }
    lane_merge_f<E>(r);
  }
}

}  // namespace tk
