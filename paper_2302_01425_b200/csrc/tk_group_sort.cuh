// tk_group_sort.cuh -- rows of up to 256 elements held by G lanes of a warp, 8
// elements per lane: load + pack, and the sorting network (19-comparator
// 8-sorter per lane, bitonic merges across lanes through shuffles).  After
// group_sort lane `lig` holds sorted ranks [8 lig, 8 lig + 8), descending.
#pragma once

#include "tk_common.cuh"

namespace tk {

constexpr int EPL = 8;   // elements per lane
__device__ __forceinline__ int pad8(int i) { return i + (i >> 3); }

__device__ __forceinline__ void ce(unsigned long long& a, unsigned long long& b) { ce_desc(a, b); }

__device__ __forceinline__ void sort8(unsigned long long (&r)[EPL]) {
  // 19-comparator network for 8 inputs (descending)
  ce(r[0], r[1]); ce(r[2], r[3]); ce(r[4], r[5]); ce(r[6], r[7]);
  ce(r[0], r[2]); ce(r[1], r[3]); ce(r[4], r[6]); ce(r[5], r[7]);
  ce(r[1], r[2]); ce(r[5], r[6]); ce(r[0], r[4]); ce(r[3], r[7]);
  ce(r[1], r[5]); ce(r[2], r[6]);
  ce(r[1], r[4]); ce(r[3], r[6]);
  ce(r[2], r[4]); ce(r[3], r[5]);
  ce(r[3], r[4]);
}

__device__ __forceinline__ void merge8(unsigned long long (&r)[EPL]) {   // bitonic -> descending
  ce(r[0], r[4]); ce(r[1], r[5]); ce(r[2], r[6]); ce(r[3], r[7]);
  ce(r[0], r[2]); ce(r[1], r[3]); ce(r[4], r[6]); ce(r[5], r[7]);
  ce(r[0], r[1]); ce(r[2], r[3]); ce(r[4], r[5]); ce(r[6], r[7]);
}

template <int G>
__device__ __forceinline__ void group_sort(unsigned long long (&r)[EPL], int lig, unsigned mask) {
  sort8(r);
#pragma unroll
  for (int size = 2; size <= G; size <<= 1) {
    {   // first stage of the merge: element g against its mirror in the block of `size` lanes
      const bool keepmax = (lig & (size >> 1)) == 0;
      unsigned long long o[EPL];
#pragma unroll
      for (int i = 0; i < EPL; ++i) o[i] = __shfl_xor_sync(mask, r[EPL - 1 - i], size - 1);
#pragma unroll
      for (int i = 0; i < EPL; ++i) r[i] = pick64(r[i], o[i], keepmax);
    }
#pragma unroll
    for (int s = size >> 2; s >= 1; s >>= 1) {
      const bool keepmax = (lig & s) == 0;
#pragma unroll
      for (int i = 0; i < EPL; ++i) {
        unsigned long long o = __shfl_xor_sync(mask, r[i], s);
        r[i] = pick64(r[i], o, keepmax);
      }
    }
    merge8(r);
  }
}

template <int G, typename T>
__device__ __forceinline__ T group_sum(T v, unsigned mask) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(mask, v, o);
  return v;
}
// exclusive prefix over the lanes of the group
template <int G>
__device__ __forceinline__ float group_excl(float v, int lig, unsigned mask) {
  float inc = v;
#pragma unroll
  for (int o = 1; o < G; o <<= 1) {
    float up = __shfl_up_sync(mask, inc, o, G);
    if (lig >= o) inc += up;
  }
  return inc - v;
}

// loads the lane's 8 consecutive elements of the row and packs them; bad: a non-finite input was seen
__device__ __forceinline__ void group_load_pack(const Problem& P, const float* x_row, int lig, bool mag,
                                                unsigned long long (&r)[EPL], bool& bad) {
  const int n = P.n;
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      int base = EPL * lig + 4 * h;
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (base < n) q = __ldg(x4 + (base >> 2));
      float e4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        if (base + c4 < n && !isfinite(e4[c4])) bad = true;
        r[4 * h + c4] = pack(e4[c4], base + c4, mag, n);
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      int idx = EPL * lig + i;
      float x = (idx < n) ? __ldg(x_row + idx) : 0.0f;
      if (idx < n && !isfinite(x)) bad = true;
      r[i] = pack(x, idx, mag, n);
    }
  }
}

}  // namespace tk
