// tk_ctav.cu -- rows of 1025..16384 elements, the default forward pass and VJP, and the forward
// pass of rows of up to 32768: one thread block per row, merge sort of the 32-bit KEYS only,
// results placed by value.  With 32 keys per thread (rows above 16384) the row itself is not
// kept in registers: the results pass reads it again (it is in L2), and the VJP is left to the
// streaming kernel that works from the saved row state.
//
// Same reasoning as tk_rows.cu: with gamma and the block edges known, the result of an element
// depends on its key alone, so no index travels through the sort (a shared-memory slot is 4 bytes,
// a comparison one instruction), nothing is scattered, and every thread stores where it loaded.
// The isotonic solve on the sorted keys is the one of tk_cta.cu (Sec. 5, App. A.6).
#include "tk_common.cuh"
#include "tk_cta_sort.cuh"
#include "tk_block_util.cuh"

namespace tk {

namespace {

struct RowSolveV { float u; };

template <int E>
__device__ __forceinline__ void sort_registers_f(float (&r)[E]) {   // bitonic network, descending
#pragma unroll
  for (int size = 2; size <= E; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const int j = i ^ stride;
        if (j > i) {
          const float hi = fmaxf(r[i], r[j]), lo = fminf(r[i], r[j]);
          if ((i & size) == 0) { r[i] = hi; r[j] = lo; } else { r[i] = lo; r[j] = hi; }
        }
      }
    }
  }
}

// The warp's 32 E keys, each lane's E already descending -> descending across the warp (lane l
// ends with ranks [l E, l E + E) of the warp's keys): bitonic merges through shuffles.
template <int E>
__device__ __forceinline__ void warp_sort_keys(float (&r)[E], int lane) {
#pragma unroll
  for (int size = 2; size <= 32; size <<= 1) {
    {
      const bool keepmax = (lane & (size >> 1)) == 0;
#pragma unroll
      for (int i = 0; i < E / 2; ++i) {            // slot i meets the partner's slot E-1-i and vice versa
        const float oa = __shfl_xor_sync(0xffffffffu, r[E - 1 - i], size - 1);
        const float ob = __shfl_xor_sync(0xffffffffu, r[i], size - 1);
        r[i] = keepmax ? fmaxf(r[i], oa) : fminf(r[i], oa);
        r[E - 1 - i] = keepmax ? fmaxf(r[E - 1 - i], ob) : fminf(r[E - 1 - i], ob);
      }
    }
#pragma unroll
    for (int st = size >> 2; st >= 1; st >>= 1) {
      const bool keepmax = (lane & st) == 0;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float o = __shfl_xor_sync(0xffffffffu, r[i], st);
        r[i] = keepmax ? fmaxf(r[i], o) : fminf(r[i], o);
      }
    }
#pragma unroll
    for (int stride = E >> 1; stride > 0; stride >>= 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const int j = i ^ stride;
        if (j > i) { const float hi = fmaxf(r[i], r[j]), lo = fminf(r[i], r[j]); r[i] = hi; r[j] = lo; }
      }
    }
  }
}

template <int E, int MAXT>
__global__ void __launch_bounds__(MAXT, MAXT == 512 ? 2 : 1)
tk_ctav_kernel(const Problem P) {
  constexpr bool KEEP = E <= 16;               // the row stays in registers for the results pass
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int T = blockDim.x;
  const int t = threadIdx.x;
  const int n = P.n, k = P.k, N = P.N;
  const long long row = blockIdx.x;
  const Math M = make_math_q24(P);
  const bool mag = M.mag;

  float* keys = reinterpret_cast<float*>(smem_raw);                              // pad(N) + 1 sorted keys
  const int key_slots = (pad(N) + 2) & ~1;
  double* cps = reinterpret_cast<double*>(keys + key_slots);                     // 3 x (T + 1)
  double* redd = cps + 3 * (T + 1);                                              // 40 doubles
  int* redi = reinterpret_cast<int*>(redd + 40);                                 // 40 ints
  __shared__ RowSolveV sol;
  __shared__ int row_flags;
  if (t == 0) row_flags = 0;

  // ---- load (striped, coalesced); x[] stays in registers for the epilogue
  const float* x_row = P.theta + row * (long long)n;
  float x[KEEP ? E : 4], s[E];
  bool bad = false;
  auto index_of = [&](int i) -> int { return P.vec4 ? 4 * ((i >> 2) * T + t) + (i & 3) : i * T + t; };
  // the thread's elements 4 j .. 4 j + 3 (zeros past the row's end)
  auto load4 = [&](const float* base, int j, float (&v4)[4]) {
    if (P.vec4) {
      const int v = j * T + t;
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (4 * v < n) q = __ldg(reinterpret_cast<const float4*>(base) + v);
      v4[0] = q.x; v4[1] = q.y; v4[2] = q.z; v4[3] = q.w;
    } else {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) { const int idx = (4 * j + c4) * T + t; v4[c4] = (idx < n) ? __ldg(base + idx) : 0.0f; }
    }
  };
  unsigned valid = 0;
#pragma unroll
  for (int j = 0; j < E / 4; ++j) {
    float v4[4];
    load4(x_row, j, v4);
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
      const int i = 4 * j + c4;
      const bool in = index_of(i) < n;
      valid |= in ? (1u << i) : 0u;
      if (in && !isfinite(v4[c4])) bad = true;
      s[i] = in ? sort_key(v4[c4], mag) : -INFINITY;      // slots past the row sort last
      if (KEEP) x[i] = v4[c4];
    }
  }

  // ---- sort of the keys: registers, the warp's 32 E keys through shuffles, then log2(T / 32)
  // merge-path rounds in shared memory
  sort_registers_f<E>(s);
  warp_sort_keys<E>(s, t & 31);
#pragma unroll
  for (int i = 0; i < E; ++i) keys[pad(t * E + i)] = s[i];
  __syncthreads();
  for (int L = 32 * E; L < N; L <<= 1) {
    const int pos = t * E;
    const int base = pos & ~(2 * L - 1);
    const int diag = pos - base;
    int lo = max(0, diag - L), hi = min(diag, L);
    for (int span = L; span > 0; span >>= 1) {             // the same number of steps in every thread
      const bool go = lo < hi;
      const int mid = go ? (lo + hi) >> 1 : 0;
      const float a = keys[pad(base + mid)];
      const float b = keys[pad(base + L + (go ? diag - 1 - mid : 0))];
      const bool up = a >= b;                              // ties: take from the first run (any order is fine)
      lo = (go && up) ? mid + 1 : lo;
      hi = (go && !up) ? mid : hi;
    }
    int ia = lo, ib = diag - lo;
    float a = (ia < L) ? keys[pad(base + ia)] : -INFINITY;
    float b = (ib < L) ? keys[pad(base + L + ib)] : -INFINITY;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      // an exhausted run can never win: -inf >= -inf only when both are (padding, whose order is free)
      const bool takeA = (ia < L) && (!(ib < L) || a >= b);
      s[i] = takeA ? a : b;
      ia += takeA ? 1 : 0;
      ib += takeA ? 0 : 1;
      const int nxt = takeA ? ia : L + ib;
      const bool in = takeA ? (ia < L) : (ib < L);
      const float v = in ? keys[pad(base + nxt)] : -INFINITY;
      a = takeA ? v : a;
      b = takeA ? b : v;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < E; ++i) keys[pad(pos + i)] = s[i];
    __syncthreads();
  }
  // thread t holds sorted ranks [tE, tE + E) in s[], keys[] holds the whole sorted row

  // ---- isotonic solve
  const float c = keys[pad(k - 1)];
  const float vtop_c = M.vtop(c);
  bool has_block = false;
  if (k < n) {
    float sk = keys[pad(k)];
    has_block = vtop_c < sk;
  }
  // Pivot for the arithmetic around the pooled block.  The block's keys lie in
  // (vtop(c), c + width(c)); when that window stays within a factor two of c the
  // pivot c makes every difference below exact.  For phi even and large lambda the
  // window reaches far below c (gamma << c); then the keys themselves are the
  // well-scaled quantity and the pivot is 0.
  const float piv = (mag && vtop_c < 0.5f * c) ? 0.0f : c;
#define TK_D(i) (s[i] - piv)

  int a0 = k, b0 = k;
  float u = 0.0f;
  if (has_block) {
    const float W_hi = (piv == c) ? M.width(c) : c + M.width(c);
    const float W_lo = vtop_c - piv;
    // window counts and chunk sums
    int c_hi = 0, c_lo = 0;
    float s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      bool valid = (t * E + i) < n;
      const float di = TK_D(i);
      bool ge_hi = valid && (di >= W_hi);
      bool gt_lo = valid && (di > W_lo);
      c_hi += ge_hi; c_lo += gt_lo;
      if (gt_lo && !ge_hi) { s1 += di; float d2 = di * di; s2 += d2; s3 += d2 * di; }
    }
    int wl, wh;
    {
      int tot;
      block_exclusive_scan<int>(c_hi, redi, &tot); wl = tot;
      block_exclusive_scan<int>(c_lo, redi, &tot); wh = tot;
    }
    {
      double tot;
      double e1 = block_exclusive_scan<double>((double)s1, redd, &tot);
      cps[t] = e1; if (t == 0) cps[T] = tot;
      if (M.q4) {
        double e2 = block_exclusive_scan<double>((double)s2, redd, &tot);
        cps[(T + 1) + t] = e2; if (t == 0) cps[(T + 1) + T] = tot;
        double e3 = block_exclusive_scan<double>((double)s3, redd, &tot);
        cps[2 * (T + 1) + t] = e3; if (t == 0) cps[2 * (T + 1) + T] = tot;
      }
    }
    __syncthreads();

    // prefix sums of d^m over window ranks below r
    auto prefix = [&](int rk, double& p1, double& p2, double& p3) {
      int ch = rk / E;
      p1 = cps[ch]; p2 = 0.0; p3 = 0.0;
      if (M.q4) { p2 = cps[(T + 1) + ch]; p3 = cps[2 * (T + 1) + ch]; }
      float f1 = 0.f, f2 = 0.f, f3 = 0.f;
      for (int i = ch * E; i < rk; ++i) {
        if (i >= wl && i < wh) {
          float di = keys[pad(i)] - piv;
          f1 += di; float q2 = di * di; f2 += q2; f3 += q2 * di;
        }
      }
      p1 += f1; p2 += f2; p3 += f3;
    };
    // F at gamma = c + uu with the ranks [r_hi, r_lo) strictly between the caps
    auto evalF = [&](float uu, int r_hi, int r_lo) -> float {
      double h1, h2, h3, l1, l2, l3;
      prefix(r_hi, h1, h2, h3);
      prefix(r_lo, l1, l2, l3);
      float cnt = (float)(r_lo - r_hi);
      float D1 = (float)(l1 - h1);
      float S;
      if (M.q4) {
        float D2 = (float)(l2 - h2), D3 = (float)(l3 - h3);
        S = (((-cnt * uu + 3.0f * D1) * uu - 3.0f * D2) * uu + D3) * (P.inv_lam * P.inv_lam * P.inv_lam);
      } else {
        S = (D1 - cnt * uu) * P.inv_lam;
      }
      if (mag) S = S / (piv + uu);
      return (float)(r_hi - k) + S;
    };
    // number of ranks in [L, R) whose d >= x (d non-increasing)
    auto count_ge = [&](float x, int L, int R) -> int {
      while (L < R) {
        int mid = (L + R) >> 1;
        float dm = keys[pad(mid)] - piv;
        if (dm >= x) L = mid + 1; else R = mid;
      }
      return L;
    };
    auto count_gt = [&](float x, int L, int R) -> int {
      while (L < R) {
        int mid = (L + R) >> 1;
        float dm = keys[pad(mid)] - piv;
        if (dm > x) L = mid + 1; else R = mid;
      }
      return L;
    };
    // predB(j): rank j lies strictly above gamma.  predA(j): rank j stays a top singleton.
    auto predB = [&](int j) -> bool {
      if (j < k) return true;
      if (j >= wh) return false;
      float tau = keys[pad(j)];
      float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      int r_hi = count_ge(uu + M.width(tau), wl, k);
      return evalF(uu, r_hi, j) < 0.0f;
    };
    auto predA = [&](int j) -> bool {
      if (j < wl) return true;
      if (j >= k) return false;
      float tau = M.vtop(keys[pad(j)]);
      float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      int r_lo = count_gt(uu, k, wh);
      return evalF(uu, j, r_lo) <= 0.0f;
    };
    // T-ary search, two rounds: chunk, then rank within the chunk
    int tb = max(__syncthreads_count(predB(t * E)) - 1, 0);
    int ta = max(__syncthreads_count(predA(t * E)) - 1, 0);
    int cb = __syncthreads_count(t < E && predB(tb * E + t));
    int ca = __syncthreads_count(t < E && predA(ta * E + t));
    b0 = tb * E + cb;
    a0 = ta * E + ca;
    b0 = min(max(b0, k + 1), wh);
    a0 = max(min(a0, k - 1), wl);

    if (t == 0) {
      double h1, h2, h3, l1, l2, l3;
      prefix(a0, h1, h2, h3);
      prefix(b0, l1, l2, l3);
      double cnt = (double)(b0 - a0), m = (double)(k - a0);
      double D1 = l1 - h1, D2 = l2 - h2, D3 = l3 - h3;
      double u_left = mag ? (double)W_lo : D1 / cnt - (double)P.lam * cbrt(m / cnt);
      int nc = 0;
      double uu = solve_block_u(M.q4, mag, (double)P.lam, (double)piv, cnt, m, D1, D2, D3, u_left, &nc);
      sol.u = settle_offset(M, piv, (float)uu, a0, b0, n, [&](int i) -> float { return keys[pad(i)]; });
      if (nc) atomicOr(&row_flags, TK_FLAG_NOT_CONVERGED);
    }
    __syncthreads();
    u = sol.u;
  }
  if (bad) atomicOr(&row_flags, TK_FLAG_NONFINITE);

  if (P.state_out && t == 0) {
    tk_rowstate st;
    st.pivot = has_block ? piv : c; st.offset = u; st.a = a0; st.b = b0;
    P.state_out[row] = st;
  }

#undef TK_D
  // ---- epilogue by value, in the original (striped) order
  const float wid = has_block ? M.width(piv + u) : 0.0f;
  auto classify = [&](float key, float& tt) -> int {      // 2 capped, 1 pooled, 0 zero
    if (!has_block) { tt = 0.0f; return key >= c ? 2 : 0; }
    const float tq = (key - piv) - u;
    tt = fminf(fmaxf(tq, 0.0f), wid);
    return tq >= wid ? 2 : (tq > 0.0f ? 1 : 0);
  };
  float* o_row = P.out + row * (long long)n;
  if constexpr (!KEEP) {
    // forward pass only; the row is read again, four elements at a time, and stored at once
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      float v4[4], o4v[4];
      load4(x_row, j, v4);
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        float tt;
        const float key = sort_key(v4[c4], mag);
        const int cls = classify(key, tt);
        float v = cls == 2 ? (mag ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
        if (mag) v = signbit(v4[c4]) ? -v : v;
        if (P.mode == TK_TOPK) v *= v4[c4];
        o4v[c4] = v;
      }
      if (P.vec4) {
        const int v = j * T + t;
        if (4 * v < n) reinterpret_cast<float4*>(o_row)[v] = make_float4(o4v[0], o4v[1], o4v[2], o4v[3]);
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) { const int idx = (4 * j + c4) * T + t; if (idx < n) o_row[idx] = o4v[c4]; }
      }
    }
  } else {
  float o[E];
  if (P.what == W_FWD) {
#pragma unroll
    for (int i = 0; i < E; ++i) {
      float tt;
      const float key = sort_key(x[i], mag);
      const int cls = classify(key, tt);
      float v = cls == 2 ? (mag ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
      if (mag) v = signbit(x[i]) ? -v : v;
      if (P.mode == TK_TOPK) v *= x[i];
      o[i] = v;
    }
  } else {
    // ---- VJP (Prop. 7), by value
    const float* g_row = P.gout + row * (long long)n;
    float g[E];
    if (P.vec4) {
#pragma unroll
      for (int j = 0; j < E / 4; ++j) {
        const int v = j * T + t;
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        if (4 * v < n) q = __ldg(reinterpret_cast<const float4*>(g_row) + v);
        g[4 * j] = q.x; g[4 * j + 1] = q.y; g[4 * j + 2] = q.z; g[4 * j + 3] = q.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < E; ++i) { const int idx = i * T + t; g[i] = (idx < n) ? __ldg(g_row + idx) : 0.0f; }
    }
    float A = 0.f, D = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      float tt;
      if (((valid >> i) & 1u) && classify(sort_key(x[i], mag), tt) == 1) {
        const float dr = M.drho(tt);
        const float chi = mag ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
        D += dr; A += dr * chi * g[i];
      }
    }
    const float Ab = block_sum<float>(A, reinterpret_cast<float*>(redd));
    float Db = block_sum<float>(D, reinterpret_cast<float*>(redd));
    if (mag) Db += (float)(k - a0);
    const float ratio = (Db > 0.0f) ? Ab / Db : 0.0f;
    // second pass: residuals about the fp32 mean (one fma each, no cancellation) restore what the
    // division rounded away; rho' can be 3/lambda, and an ulp of the mean times that shows
    float A2 = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      float tt;
      if (((valid >> i) & 1u) && classify(sort_key(x[i], mag), tt) == 1) {
        const float chi = mag ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
        A2 += M.drho(tt) * fmaf(chi, g[i], -ratio);
      }
    }
    float A2b = block_sum<float>(A2, reinterpret_cast<float*>(redd));
    if (mag) A2b -= (float)(k - a0) * ratio;
    const float delta = (Db > 0.0f) ? A2b / Db : 0.0f;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      float tt;
      const float key = sort_key(x[i], mag);
      const int cls = classify(key, tt);
      const float sgn = (mag && signbit(x[i])) ? -1.0f : 1.0f;
      const float chi = mag ? sgn : (P.mode == TK_TOPK ? x[i] : 1.0f);
      float v = 0.0f;
      if (cls == 1) v = M.drho(tt) * (fmaf(chi, g[i], -ratio) - delta);
      else if (cls == 2 && mag) v = chi * g[i] * M.top_slope(key);
      v *= sgn;
      if (P.mode == TK_TOPK) v += g[i] * (cls == 2 ? 1.0f : (cls == 1 ? M.rho(tt) : 0.0f));
      o[i] = v;
    }
  }
  if (P.vec4) {
    float4* o4 = reinterpret_cast<float4*>(o_row);
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int v = j * T + t;
      if (4 * v < n) o4[v] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i) { const int idx = i * T + t; if (idx < n) o_row[idx] = o[i]; }
  }
  }   // KEEP
  if (t == 0 && row_flags && P.status) atomicOr(P.status, row_flags);
}

}  // namespace

int cta_padded_length(int n);

// rows of up to 16384: forward pass or recomputing VJP; up to 32768: forward pass only
cudaError_t launch_ctav(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  P.N = cta_padded_length(P.n);
  if (P.N < 512) P.N = 512;
  // one warp sorts 32 E keys; T = N / E threads.  32 keys per thread (forward pass only) from 16384
  // elements: 512 threads per row there, and the only way to hold 32768
  const int E = (P.N > 16384 || (P.N >= 2048 && P.what == W_FWD)) ? 32 : 16;
  if (E == 32 && P.what != W_FWD) return cudaErrorInvalidValue;
  const int T = P.N / E;
  const size_t smem = (size_t)(((P.N + (P.N >> PAD_SHIFT)) + 2) & ~1) * 4 + (size_t)3 * (T + 1) * 8 + 40 * 8 + 40 * 4 + 64;
  void (*kern)(const Problem) = nullptr;
  int slot;
  if (E == 32 && T <= 512) { kern = tk_ctav_kernel<32, 512>; slot = 3; }
  else if (E == 32) { kern = tk_ctav_kernel<32, 1024>; slot = 0; }
  else if (T > 512) { kern = tk_ctav_kernel<16, 1024>; slot = 2; }
  else { kern = tk_ctav_kernel<16, 512>; slot = 1; }
  static bool configured[4][64] = {};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !configured[slot][dev]) {
    const int max_n = (slot == 0) ? 32768 : 16384;
    const int max_smem = (max_n + (max_n >> PAD_SHIFT) + 2) * 4 + 3 * 1025 * 8 + 40 * 8 + 40 * 4 + 64;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) configured[slot][dev] = true;
  }
  kern<<<(unsigned)P.rows, (unsigned)T, smem, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace tk
