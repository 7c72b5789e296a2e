// tk_group_sort.cuh -- rows held by G lanes of a warp, E = 8 or 16 elements per
// lane (up to 512 elements): load + pack, and the sorting network (19-comparator
// 8-sorter per lane, bitonic merges inside the lane and across lanes through
// shuffles).  After group_sort lane `lig` holds sorted ranks [E lig, E lig + E),
// descending.
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

// shared-memory index of rank i when every lane owns E consecutive ranks: one spare slot per E
template <int E>
__device__ __forceinline__ int pad_e(int i) { return i + (i / E); }

// descending sort of the lane's E registers
template <int E>
__device__ __forceinline__ void lane_sort(unsigned long long (&r)[E]);
template <>
__device__ __forceinline__ void lane_sort<8>(unsigned long long (&r)[8]) { sort8(r); }
// bitonic sequence in the lane's E registers -> descending
template <int E>
__device__ __forceinline__ void lane_merge(unsigned long long (&r)[E]);
template <>
__device__ __forceinline__ void lane_merge<8>(unsigned long long (&r)[8]) { merge8(r); }
template <>
__device__ __forceinline__ void lane_merge<16>(unsigned long long (&r)[16]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) ce(r[i], r[i + 8]);
  unsigned long long lo[8], hi[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { hi[i] = r[i]; lo[i] = r[i + 8]; }
  merge8(hi); merge8(lo);
#pragma unroll
  for (int i = 0; i < 8; ++i) { r[i] = hi[i]; r[i + 8] = lo[i]; }
}
template <>
__device__ __forceinline__ void lane_sort<16>(unsigned long long (&r)[16]) {
  unsigned long long hi[8], lo[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { hi[i] = r[i]; lo[i] = r[i + 8]; }
  sort8(hi); sort8(lo);
  // merge two descending runs: element i against its mirror, then each half is bitonic
#pragma unroll
  for (int i = 0; i < 8; ++i) ce(hi[i], lo[7 - i]);
  merge8(hi); merge8(lo);
#pragma unroll
  for (int i = 0; i < 8; ++i) { r[i] = hi[i]; r[i + 8] = lo[i]; }
}

template <int G, int E>
__device__ __forceinline__ void group_sort_e(unsigned long long (&r)[E], int lig, unsigned mask) {
  lane_sort<E>(r);
#pragma unroll
  for (int size = 2; size <= G; size <<= 1) {
    {   // first stage of the merge: element g against its mirror in the block of `size` lanes
      const bool keepmax = (lig & (size >> 1)) == 0;
      unsigned long long o[E];
#pragma unroll
      for (int i = 0; i < E; ++i) o[i] = __shfl_xor_sync(mask, r[E - 1 - i], size - 1);
#pragma unroll
      for (int i = 0; i < E; ++i) r[i] = pick64(r[i], o[i], keepmax);
    }
#pragma unroll
    for (int s = size >> 2; s >= 1; s >>= 1) {
      const bool keepmax = (lig & s) == 0;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        unsigned long long o = __shfl_xor_sync(mask, r[i], s);
        r[i] = pick64(r[i], o, keepmax);
      }
    }
    lane_merge<E>(r);
  }
}
template <int G>
__device__ __forceinline__ void group_sort(unsigned long long (&r)[EPL], int lig, unsigned mask) {
  group_sort_e<G, EPL>(r, lig, mask);
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

// loads the lane's E consecutive elements of the row and packs them; bad: a non-finite input was seen
template <int E>
__device__ __forceinline__ void group_load_pack_e(const Problem& P, const float* x_row, int lig, bool mag,
                                                  unsigned long long (&r)[E], bool& bad) {
  const int n = P.n;
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
#pragma unroll
    for (int h = 0; h < E / 4; ++h) {
      int base = E * lig + 4 * h;
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
    for (int i = 0; i < E; ++i) {
      int idx = E * lig + i;
      float x = (idx < n) ? __ldg(x_row + idx) : 0.0f;
      if (idx < n && !isfinite(x)) bad = true;
      r[i] = pack(x, idx, mag, n);
    }
  }
}
__device__ __forceinline__ void group_load_pack(const Problem& P, const float* x_row, int lig, bool mag,
                                                unsigned long long (&r)[EPL], bool& bad) {
  group_load_pack_e<EPL>(P, x_row, lig, mag, r, bad);
}

}  // namespace tk
