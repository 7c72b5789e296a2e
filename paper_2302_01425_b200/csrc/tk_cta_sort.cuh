// tk_cta_sort.cuh -- one thread block per row: load + pack, register bitonic
// sort of each thread's E elements, then log2(T) merge-path rounds in padded
// shared memory.  On return thread t holds sorted ranks [tE, tE + E) in r[]
// (descending) and keys[pad(i)] holds rank i for the whole row.
#pragma once

#include "tk_common.cuh"

namespace tk {

constexpr int PAD_SHIFT = 4;   // one spare 8-byte slot every 16 keeps blocked accesses conflict-free
__device__ __forceinline__ int pad(int i) { return i + (i >> PAD_SHIFT); }

template <int E>
__device__ __forceinline__ void sort_registers(unsigned long long (&r)[E]) {
  // bitonic network, fully unrolled, descending
#pragma unroll
  for (int size = 2; size <= E; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        int j = i ^ stride;
        if (j > i) {
          if ((i & size) == 0) ce_desc(r[i], r[j]); else ce_desc(r[j], r[i]);
        }
      }
    }
  }
}

template <int E>
__device__ __forceinline__ void cta_load_sort(const Problem& P, const float* x_row, unsigned long long* keys,
                                              unsigned long long (&r)[E], bool& bad) {
  const int T = blockDim.x, t = threadIdx.x, n = P.n, N = P.N;
  const bool mag = P.mode == TK_TOPKMAG;
  // ---- load (striped, coalesced) and pack
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      int v = j * T + t;
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (4 * v < n) q = __ldg(x4 + v);
      float e4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        int idx = 4 * v + c4;
        if (idx < n && !isfinite(e4[c4])) bad = true;
        r[4 * j + c4] = pack(e4[c4], idx, mag, n);
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i) {
      int idx = i * T + t;
      float x = (idx < n) ? __ldg(x_row + idx) : 0.0f;
      if (idx < n && !isfinite(x)) bad = true;
      r[i] = pack(x, idx, mag, n);
    }
  }

  // ---- sort: registers, then log2(T) merge rounds through shared memory
  sort_registers<E>(r);
#pragma unroll
  for (int i = 0; i < E; ++i) keys[pad(t * E + i)] = r[i];
  __syncthreads();
  for (int L = E; L < N; L <<= 1) {
    const int pos = t * E;                   // first output position of this thread
    const int base = pos & ~(2 * L - 1);
    const int diag = pos - base;
    const unsigned long long* A = keys;      // run A = [base, base+L), run B = [base+L, base+2L)
    int lo = max(0, diag - L), hi = min(diag, L);
    // merge path: the same number of halving steps in every thread (no divergence)
    for (int span = L; span > 0; span >>= 1) {
      const bool go = lo < hi;
      const int mid = go ? (lo + hi) >> 1 : 0;
      const int ib_probe = go ? diag - 1 - mid : 0;
      const unsigned long long a = A[pad(base + mid)];
      const unsigned long long b = A[pad(base + L + ib_probe)];
      const bool up = a > b;
      lo = (go && up) ? mid + 1 : lo;
      hi = (go && !up) ? mid : hi;
    }
    int ia = lo, ib = diag - lo;
    unsigned long long a = (ia < L) ? A[pad(base + ia)] : 0ull;
    unsigned long long b = (ib < L) ? A[pad(base + L + ib)] : 0ull;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const bool takeA = a > b;
      r[i] = sel64(takeA, a, b);
      ia += takeA ? 1 : 0;
      ib += takeA ? 0 : 1;
      const int nxt = takeA ? ia : L + ib;                 // one load per step, from the run that advanced
      const bool in = takeA ? (ia < L) : (ib < L);
      const unsigned long long v = in ? A[pad(base + nxt)] : 0ull;
      a = sel64(takeA, v, a);
      b = sel64(takeA, b, v);
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < E; ++i) keys[pad(pos + i)] = r[i];
    __syncthreads();
  }
}

}  // namespace tk
