// tk_thr.cu -- the exact forward pass without a sort, one thread block per row: the solver for a general
// p (1 < p < 2 other than 4/3).  p = 2 and p = 4/3 take the register-resident team kernel of
// tk_newton.cu; the closed-form variants of this kernel (QM = 0, 1) are kept as templates but not launched.
//
// With w = 1_k the isotonic solution has at most one pooled block, whose value
// gamma is the root of the non-increasing threshold function
//   F(tau) = #{key_i >= tau + width(tau)} + sum_{tau < key_i < tau + width} rho(key_i - tau)/phi'(tau) - k
// (Sec. 3: the mask is the maximiser over the capped simplex; its stationarity
// condition in the threshold form).  Nothing in F needs the order of the keys:
//   1. radix-select the k-th largest key c exactly (four 8-bit histogram passes
//      over the order-preserving integer keys), then the largest key below it:
//      the same no-block test vtop(c) >= s_k as the sorted path;
//   2. safeguarded Newton on F inside the bracket (vtop(c), s_k): every pass
//      classifies the row against tau (capped / strictly inside / zero), sums
//      the inside keys relative to tau, and solves the stationarity equation of
//      that candidate set in closed form (p = 2) or by the App. A.6 cubic
//      (p = 4/3); when the candidate reproduces its own set the root is exact --
//      it is the value pool-adjacent-violators ends with (Sec. 5);
//   3. dual map in the original order: no permutation, no scatter.
// One thread block per row, the row in registers.  The row state written for the
// VJP has the format of the sorted path (gamma = pivot + offset).
#include "tk_common.cuh"

namespace tk {

namespace {

struct Sums {
  int ct, cm;          // capped (top) and strictly-inside counts
  float s1, s2, s3;    // sums of t, t^2, t^3 over the inside keys, t = key - tau
                       // (any other q: s1 = sum rho(t), s2 = sum rho'(t))
};

// block-wide sum of the five accumulators; result in every thread.  red: 5 x 32 floats
__device__ __forceinline__ Sums block_reduce(Sums v, float* red, bool q4) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v.ct = warp_sum(v.ct); v.cm = warp_sum(v.cm); v.s1 = warp_sum(v.s1);
  if (q4) { v.s2 = warp_sum(v.s2); v.s3 = warp_sum(v.s3); }
  if (lane == 0) {
    red[warp] = __int_as_float(v.ct); red[32 + warp] = __int_as_float(v.cm); red[64 + warp] = v.s1;
    red[96 + warp] = v.s2; red[128 + warp] = v.s3;
  }
  __syncthreads();
  Sums r;
  int a = (lane < nw) ? __float_as_int(red[lane]) : 0, b = (lane < nw) ? __float_as_int(red[32 + lane]) : 0;
  float c1 = (lane < nw) ? red[64 + lane] : 0.f;
  r.ct = warp_sum(a); r.cm = warp_sum(b); r.s1 = warp_sum(c1); r.s2 = 0.f; r.s3 = 0.f;
  if (q4) {
    float c2 = (lane < nw) ? red[96 + lane] : 0.f, c3 = (lane < nw) ? red[128 + lane] : 0.f;
    r.s2 = warp_sum(c2); r.s3 = warp_sum(c3);
  }
  __syncthreads();
  return r;
}

// Step du that solves the candidate set's cubic (App. A.6) with the sums taken about the current
// gamma:  sum (t_i - du)^3 = lam^3 m [(gamma + du) for phi even].  Because the anchor is the
// current iterate, du -> 0 as the outer iteration converges and fp32 is enough: an error of one
// ulp of S3 moves du by about 1e-7 of the block's width, and the next pass re-anchors.
__device__ __forceinline__ float solve_piece_cubic(bool mag, float lam3, float gam, float cnt, float m,
                                                   float S1, float S2, float S3) {
  const float l3m = lam3 * m;
  const float mu = S1 / cnt;
  const float m2 = fmaxf(S2 - S1 * mu, 0.0f);
  const float m3 = S3 - 3.0f * mu * S2 + 2.0f * mu * mu * S1;
  const float Pc = (3.0f * m2 + (mag ? l3m : 0.0f)) / cnt;
  const float Qc = (l3m * (mag ? (gam + mu) : 1.0f) - m3) / cnt;
  const float third = Pc * (1.0f / 3.0f);
  const float R = sqrtf(0.25f * Qc * Qc + third * third * third);
  const float A = cbrtf(0.5f * fabsf(Qc) + R);
  const float B = (A != 0.0f) ? third / A : 0.0f;
  const float den = A * A + third + B * B;
  float u = mu + ((den > 0.0f) ? -Qc / den : 0.0f);
  if (!isfinite(u)) u = 0.0f;
#pragma unroll 1
  for (int it = 0; it < 12; ++it) {
    const float g = ((-cnt * u + 3.0f * S1) * u - 3.0f * S2) * u + S3 - (mag ? l3m * (gam + u) : l3m);
    const float gp = -3.0f * ((cnt * u - 2.0f * S1) * u + S2) - (mag ? l3m : 0.0f);
    if (!(gp < 0.0f)) break;
    const float du = -g / gp;
    u += du;
    if (fabsf(du) <= 2e-7f * (fabsf(u) + (mag ? gam : 0.0f)) + 1e-37f) break;
  }
  return u;
}

// QM: 0 for q = 2, 1 for q = 4 (closed-form / cubic solve of every candidate set), 2 for any other
// q > 2 (Sec. 7, sensitivity to p: one Newton step on the candidate set's equation per pass).
template <int E, int MAXT, int QM, bool MAG>
__global__ void __launch_bounds__(MAXT) tk_thr_kernel(const Problem P) {
  constexpr bool Q4 = QM == 1, GEN = QM == 2;
  __shared__ int whist[MAXT / 32][256];   // per-warp digit counts (no contention between warps)
  __shared__ int hist[256];
  __shared__ float red[160];
  __shared__ int sh_digit, sh_kk, sh_eq;
  const int T = blockDim.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int n = P.n, k = P.k;
  const long long row = blockIdx.x;
  Math M = make_math(P);
  M.q4 = Q4; M.mag = MAG; M.gen = GEN;          // compile-time constants from here on
  constexpr bool mag = MAG;
  const float* x_row = P.theta + row * (long long)n;
  float x[E];
  bool bad = false;
  // ---- load (striped, coalesced); slots past the row hold NaN and never take part
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int v = j * T + t;
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (4 * v < n) q = __ldg(x4 + v);
      x[4 * j] = q.x; x[4 * j + 1] = q.y; x[4 * j + 2] = q.z; x[4 * j + 3] = q.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i) { const int idx = i * T + t; x[i] = (idx < n) ? __ldg(x_row + idx) : 0.0f; }
  }
  auto index_of = [&](int i) -> int { return P.vec4 ? 4 * ((i >> 2) * T + t) + (i & 3) : i * T + t; };
  // keys once; slots past the end of the row become NaN, which fails every comparison below
  float key[E];
  unsigned valid = 0;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const bool in = index_of(i) < n;
    if (in && !isfinite(x[i])) bad = true;
    valid |= in ? (1u << i) : 0u;
    key[i] = in ? sort_key(x[i], mag) : __int_as_float(0x7fc00000);
  }

  // ---- 1. the k-th largest key, exactly: MSB-first radix select on the integer keys
  uint32_t prefix = 0, pmask = 0;
  int kk = k;                                   // rank wanted among the keys matching the prefix
#pragma unroll 1
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = lane; i < 256; i += 32) whist[warp][i] = 0;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const uint32_t u = f2key(key[i]);
      const bool take = ((valid >> i) & 1u) && (u & pmask) == prefix;
      // lanes with the same digit are counted by their first lane, in the warp's own histogram
      const unsigned digit = take ? ((u >> shift) & 255u) : 256u;
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      if (take && lane == __ffs(peers) - 1) whist[warp][digit] += __popc(peers);
      __syncwarp();
    }
    __syncthreads();
    for (int i = t; i < 256; i += T) {
      int s = 0;
      for (int w2 = 0; w2 < (T >> 5); ++w2) s += whist[w2][i];
      hist[i] = s;
    }
    __syncthreads();
    if (warp == 0) {                            // lane l owns digits 255 - 8 l - j, j = 0..7 (descending)
      int h[8], s = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { h[j] = hist[255 - 8 * lane - j]; s += h[j]; }
      int inc = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { int up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
      const int before = inc - s;               // keys with a larger digit than any of this lane's
      if (before < kk && kk <= inc) {
        int run = before;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (run < kk && kk <= run + h[j]) { sh_digit = 255 - 8 * lane - j; sh_kk = kk - run; sh_eq = h[j]; }
          run += h[j];
        }
      }
    }
    __syncthreads();
    prefix |= (uint32_t)sh_digit << shift;
    pmask |= 255u << shift;
    kk = sh_kk;
    __syncthreads();
  }
  const float c = key2f(prefix);               // k-th largest key
  const int n_eq = sh_eq;                      // keys equal to c
  const int n_gt = k - kk;                     // keys strictly larger than c
  // (k+1)-th largest key: c itself when the tie reaches past rank k, else the largest key below c
  float s_k = c;
  if (n_gt + n_eq <= k) {
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      if (key[i] < c) m = fmaxf(m, key[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = (lane < (T >> 5)) ? red[lane] : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    s_k = m;
    __syncthreads();
  }
  const float vtop_c = M.vtop(c);
  const bool has_block = (k < n) && (vtop_c < s_k);

  // ---- 2. safeguarded Newton on F in (vtop(c), s_k).  gamma = piv + off with a fixed pivot
  // (the k-th largest key, or 0 when the bracket reaches far below it) so that key - gamma is
  // formed as (key - piv) - off: exact differences first, a small offset second.
  const float piv = (mag && vtop_c < 0.5f * c) ? 0.0f : c;
  float off = 0.0f;
  int a0 = k, b0 = k, flags = 0;
  if (has_block) {
    float lo = vtop_c - piv, hi = s_k - piv;   // offsets with F >= 0 at lo, F <= 0 at hi
    off = 0.5f * (lo + hi);
    int prev_ct = -1, prev_cm = -1;
    bool done = false;
#pragma unroll 1
    for (int it = 0; it < 64 && !done; ++it) {
      const float gam = piv + off;
      const float w = M.width(gam);
      Sums acc{0, 0, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float tt = (key[i] - piv) - off;      // NaN for slots past the row: neither top nor mid
        const bool top = tt >= w;
        const bool mid = tt > 0.0f && !top;
        acc.ct += top; acc.cm += mid;
        if (mid) {
          if (GEN) { acc.s1 += M.rho(tt); acc.s2 += M.drho(tt); }
          else { acc.s1 += tt; if (M.q4) { const float t2 = tt * tt; acc.s2 += t2; acc.s3 += t2 * tt; } }
        }
      }
      const Sums S = block_reduce(acc, red, Q4 || GEN);
      // every thread runs the same scalar logic on the same numbers
      const int m = k - S.ct;                  // inside keys that must carry weight
      float Fv;                                // sign of F(gamma)
      if (S.cm == 0) Fv = (float)(S.ct - k);
      else {
        const float rs = GEN ? S.s1 : (M.q4 ? S.s3 * (P.inv_lam * P.inv_lam * P.inv_lam) : S.s1 * P.inv_lam);
        Fv = (float)(S.ct - k) + (mag ? rs / gam : rs);
      }
      float du = 0.0f;
      bool have_cand = false;
      if (S.cm > 0 && m >= 1) {
        if (GEN) {
          // Newton on sum rho(t_i - du) = m about du = 0 (the sums are taken at the current gamma)
          // phi even: sum rho(t_i - du) = m (gamma + du)
          du = mag ? (S.s1 - (float)m * gam) / (S.s2 + (float)m) : (S.s2 > 0.0f ? (S.s1 - (float)m) / S.s2 : 0.0f);
        } else if (M.q4) {
          du = solve_piece_cubic(mag, P.lam3, gam, (float)S.cm, (float)m, S.s1, S.s2, S.s3);
        } else {
          const float fm = (float)m, fc = (float)S.cm;
          du = mag ? (S.s1 - P.lam * fm * gam) / (fc + P.lam * fm) : (S.s1 - P.lam * fm) / fc;
        }
        have_cand = true;
        // Exact root: this point was the solution of the previous set, it sees the same set, and
        // it already solves it (the remaining step is rounding-sized, so applying it cannot move
        // gamma across a key or a cap).
        const float scale = mag ? gam : P.lam;
        if (S.ct == prev_ct && S.cm == prev_cm && fabsf(du) <= 1e-6f * scale) {
          a0 = S.ct; b0 = S.ct + S.cm; off += du; done = true;
        }
      }
      if (!done) {
        if (Fv > 0.0f) lo = fmaxf(lo, off); else hi = fminf(hi, off);
        const float cand = off + du;
        const bool inside = have_cand && cand > lo && cand < hi && (it & 7) != 7;
        prev_ct = inside ? S.ct : -1; prev_cm = inside ? S.cm : -1;
        const float next = inside ? cand : 0.5f * (lo + hi);
        if (next == off || !(hi > lo)) {           // bracket exhausted at fp32 resolution of the offset
          a0 = S.ct; b0 = S.ct + S.cm; if (have_cand) off += du;
          done = true;
        } else {
          off = next;
        }
      }
    }
    if (!done) flags |= TK_FLAG_NOT_CONVERGED;
    {
      // The block is what the FINAL offset classifies as pooled: the row state then agrees, rank for
      // rank, with the by-value classes of the results pass below and of the VJP from state.  The
      // last step, however small, can carry an edge key across gamma or across the cap (a pooled key
      // whose rho is 1 - 1e-7 sits a few 1e-9 inside the cap): when the classes at the final offset
      // are not the set that was solved, the offset moves by single ulps towards it, a few times.
      const int want_ct = a0, want_all = b0;
#pragma unroll 1
      for (int tries = 0; tries < 5; ++tries) {
        const float w = M.width(piv + off);
        int ct = 0, cm = 0;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          const float tt = (key[i] - piv) - off;
          const bool top = tt >= w;
          ct += top; cm += (tt > 0.0f && !top);
        }
        Sums acc{ct, cm, 0.f, 0.f, 0.f};
        const Sums S = block_reduce(acc, red, false);
        a0 = S.ct; b0 = S.ct + S.cm;
        const bool up = a0 > want_ct || b0 > want_all;        // a key too many reads capped / pooled
        const bool down = a0 < want_ct || b0 < want_all;
        if (up == down || tries == 4 || !done) break;
        off = nextafterf(off, up ? INFINITY : -INFINITY);
      }
    }
    if (b0 <= a0) { a0 = k; b0 = k; }              // degenerate end of the bracket search: treat as no block
  }
  const bool block = b0 > a0;
  if (P.state_out && t == 0) {
    tk_rowstate st;
    st.pivot = block ? piv : c; st.offset = block ? off : 0.0f; st.a = a0; st.b = b0;
    P.state_out[row] = st;
  }

  // ---- 3. dual map, in place
  const float wid = block ? M.width(piv + off) : 0.0f;
  float* o_row = P.out + row * (long long)n;
  float y[E];
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const float kx = key[i];
    float v;
    if (block) {
      const float tt = (kx - piv) - off;
      if (tt >= wid) v = mag ? M.vtop(kx) : 1.0f;
      else if (tt > 0.0f) v = M.rho(tt);
      else v = 0.0f;
    } else {
      v = (kx >= c) ? (mag ? M.vtop(kx) : 1.0f) : 0.0f;
    }
    if (mag) v = signbit(x[i]) ? -v : v;
    if (P.mode == TK_TOPK) v *= x[i];
    y[i] = v;
  }
  if (P.vec4) {
    float4* o4 = reinterpret_cast<float4*>(o_row);
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const int v = j * T + t;
      if (4 * v < n) o4[v] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < E; ++i) { const int idx = i * T + t; if (idx < n) o_row[idx] = y[i]; }
  }
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
  if (flags && P.status && t == 0) atomicOr(P.status, flags);
}

}  // namespace

cudaError_t launch_thr(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  int N = 128;
  while (N < P.n) N <<= 1;
  P.N = N;
  // threads: 32..1024, a multiple of 32; items per thread 4, 8 or 16
  const int E = N >= 4096 ? 16 : (N >= 1024 ? 8 : 4);
  const int T = N / E;
  const dim3 grid((unsigned)P.rows);
  // p = 2 and p = 4/3 are served by the register-resident team kernel (tk_newton.cu); this block-per-row
  // solver is launched for a general p only
  if (!(P.qm1 > 0.0f)) return cudaErrorInvalidValue;
  const bool mag = P.mode == TK_TOPKMAG;
#define TK_THR_LAUNCH(EE, MT)                                                        \
  do {                                                                               \
    if (mag) tk_thr_kernel<EE, MT, 2, true><<<grid, T, 0, stream>>>(P);               \
    else tk_thr_kernel<EE, MT, 2, false><<<grid, T, 0, stream>>>(P);                  \
  } while (0)
  switch (E) {
    case 4: TK_THR_LAUNCH(4, 128); break;
    case 8: TK_THR_LAUNCH(8, 256); break;
    default: TK_THR_LAUNCH(16, 1024); break;
  }
#undef TK_THR_LAUNCH
  return cudaGetLastError();
}

}  // namespace tk
