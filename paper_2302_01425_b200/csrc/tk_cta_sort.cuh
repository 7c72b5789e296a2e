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
          bool desc = (i & size) == 0;
          unsigned long long a = r[i], b = r[j];
          bool sw = desc ? (a < b) : (a > b);
          r[i] = sw ? b : a;
          r[j] = sw ? a : b;
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
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      unsigned long long a = A[pad(base + mid)];
      unsigned long long b = A[pad(base + L + diag - 1 - mid)];
      if (a > b) lo = mid + 1; else hi = mid;
    }
    int ia = lo, ib = diag - lo;
    unsigned long long a = (ia < L) ? A[pad(base + ia)] : 0ull;
    unsigned long long b = (ib < L) ? A[pad(base + L + ib)] : 0ull;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      bool takeA = a > b;
      r[i] = takeA ? a : b;
      if (takeA) { ++ia; a = (ia < L) ? A[pad(base + ia)] : 0ull; }
      else       { ++ib; b = (ib < L) ? A[pad(base + L + ib)] : 0ull; }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < E; ++i) keys[pad(pos + i)] = r[i];
    __syncthreads();
  }
}

}  // namespace tk
