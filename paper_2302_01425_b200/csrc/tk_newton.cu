// tk_newton.cu -- the exact forward pass without a sort, for phi(x) = x (TK_MASK, TK_TOPK),
// p = 2 and p = 4/3, rows of up to 4096 elements held in registers.
//
// With w = 1_k the relaxed mask is the maximiser of <y, x> - R(y) over the capped simplex
// P(1_k) = {y in [0,1]^n, sum y = k} (Sec. 3), so y_i = clip(rho(x_i - tau), 0, 1) with tau the
// root of the non-increasing function
//   F(tau) = #{x_i - tau >= lambda} + sum_{0 < x_i - tau < lambda} rho(x_i - tau) - k.
// That root is the value gamma of the single pooled block pool-adjacent-violators ends with
// (Sec. 5), the elements strictly inside (gamma, gamma + lambda) are its members, those above it
// the top singletons.  F is piecewise linear (p = 2) or piecewise cubic (p = 4/3); on one piece
// it is the stationarity equation of that piece's candidate block (the example of Sec. 5, the
// cubic of App. A.6), solved here from the piece's power sums.  The iteration is Newton's on
// the pieces, inside a bracket that every evaluated point tightens:
//   - start: tau0 = mean + z std - lambda (1 - 1/q), z the normal quantile of 1 - k/n (a guess,
//     nothing depends on the data being Gaussian); for k <= 2 the k+1 largest keys are tracked
//     exactly instead, which gives the bracket (s_k - lambda, s_{k+1}) or "no block" at once;
//   - one pass over the registers classifies the row against tau (capped / inside / zero) and
//     sums t, t^2, t^3 over the inside keys; the piece's equation gives the next tau;
//   - a step that leaves the bracket is replaced by a step of doubling length towards the root,
//     then by bisection (of the ordered integer keys when the bracket spans many binades), and
//     after six Newton steps in a row one such step is forced: the loop ends;
//   - the root is accepted when a point reproduces the set of the pass before it and already
//     solves it to rounding, or when cm |du| is rounding-sized (F has slope >= 1/lambda until
//     it reaches an integer, so the root is then within that distance).
// tau is kept as pivot + offset, keys as d = x - pivot, so that t = d - offset is formed without
// cancellation; the row state stores exactly the pair the last pass classified with, and its
// counts, so the VJP from state sees the same classes.
//
// Layout: G lanes of a warp per row (32/G rows per warp), E keys per lane.  The warp's rows are
// contiguous in memory: they are staged through a shared-memory tile with coalesced 128-bit
// accesses, every lane reads its own span from the tile (chunk order rotated per lane: no bank
// conflicts), results go back through the tile the same way.
#include <math.h>

#include "tk_common.cuh"

namespace tk {

namespace {

constexpr int kNtWarps = 4;               // warps per thread block
constexpr int kNtThreads = kNtWarps * 32;
constexpr int kNtMaxPasses = 200;

// rotation of the chunk order that makes the per-lane float4 reads of a quarter warp hit 8 bank groups
template <int E>
__device__ __forceinline__ int nt_rot(int lane) {
  constexpr int CH = E / 4;
  return CH >= 8 ? lane : (lane * CH) >> 3;
}

template <int G>
__device__ __forceinline__ float nt_gsum(float v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int G>
__device__ __forceinline__ int nt_gsum(int v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int G>
__device__ __forceinline__ float nt_gmax(float v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
template <int G>
__device__ __forceinline__ float nt_gmin(float v) {
#pragma unroll
  for (int o = G >> 1; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// keeps (m1 >= m2 >= m3) the three largest values seen
__device__ __forceinline__ void nt_top3(float x, float& m1, float& m2, float& m3) {
  float r = fminf(m1, x);
  m1 = fmaxf(m1, x);
  float r2 = fminf(m2, r);
  m2 = fmaxf(m2, r);
  m3 = fmaxf(m3, r2);
}

// Root of g(u) = sum_i (t_i - u)^3 - rhs (rhs >= 0) over the cm inside keys, from their power sums.
// g is decreasing; by Jensen g(mu - cbrt(rhs / cm)) >= 0 with mu the mean of the t_i, so that point is
// left of the root, where g is convex: Newton from it increases monotonically to the root.  The
// anchor of the sums is the current iterate, so u -> 0 as the outer iteration converges and fp32
// is enough.  c0 = g(0).
__device__ __forceinline__ float nt_cubic(int cm, float s1, float s2, float s3, float rhs, float c0) {
  const float fcm = (float)cm;
  const float mu = s1 / fcm;
  float u = mu - cbrtf(rhs / fcm);
  const float spread = sqrtf(s2 / fcm);
#pragma unroll 1
  for (int it = 0; it < 8; ++it) {
    const float g = ((-fcm * u + 3.0f * s1) * u - 3.0f * s2) * u + c0;
    const float gp = -3.0f * ((fcm * u - 2.0f * s1) * u + s2);
    if (!(gp < 0.0f)) break;
    const float st = -g / gp;
    u += st;
    if (fabsf(st) <= 1e-7f * (fabsf(u) + spread)) break;
  }
  return u;
}

struct NtRow {
  float piv, off;            // tau = piv + off
  float lo_o, hi_o;          // bracket of the offset: F > 0 at lo_o, F <= 0 at hi_o
  float lo_a, hi_a;          // the same bracket as absolute values of tau
  int prev_ct, prev_cm;      // classes of the pass before
  int gallop, nnewt;
  bool edge_tried;
  int a0, b0;
  bool done, noblock, repiv;
};

// What one pass found at S.off -> the next offset, or the end of the iteration.
template <bool Q4>
__device__ __forceinline__ void nt_step(NtRow& S, int ct, int cm, float s1, float s2, float s3, int k,
                                        float lam, float lam3, float tol) {
  const float wid = lam;
  S.repiv = false;
  const int m = k - ct;                        // weight the inside keys have to carry
  if (cm == 0 && ct == k) {                    // F = 0 on a flat piece: no pooled block
    S.noblock = true; S.done = true; S.a0 = k; S.b0 = k;
    return;
  }
  // more than k keys capped: no piece to solve, the root is further right by an unknown amount
  const bool have = cm > 0 && m >= 0;
  float du = 0.0f;
  bool fpos;                                   // F(tau) > 0: the root is to the right
  if (have) {
    float c0;
    if (!Q4) {
      c0 = s1 - lam * (float)m;
      du = c0 / (float)cm;
    } else {
      const float rhs = lam3 * (float)m;
      c0 = s3 - rhs;
      du = nt_cubic(cm, s1, s2, s3, rhs, c0);
      if ((du > 0.0f) != (c0 > 0.0f)) du = c0 / (3.0f * s2);
    }
    fpos = c0 > 0.0f;
    const float adu = fabsf(du);
    // a pooled block has members of both weights: 1 <= m < cm
    if (adu <= tol && m >= 1 && m < cm &&
        ((ct == S.prev_ct && cm == S.prev_cm) || (float)cm * adu <= tol)) {
      S.done = true; S.a0 = ct; S.b0 = ct + cm;
      return;
    }
  } else {
    fpos = ct >= k;                            // ct == k here means cm > 0: F > 0
  }
  S.prev_ct = ct; S.prev_cm = cm;
  if (fpos) { S.lo_o = S.off; S.lo_a = S.piv + S.off; } else { S.hi_o = S.off; S.hi_a = S.piv + S.off; }
  bool ok = false;
  float nxt = S.off;
  float cand = S.off;
  if (have) {
    cand = S.off + du;
    // every inside key would have to reach the cap: aim just past it, so that they read as capped
    if (m == cm) cand -= 0.5f * tol;
    ok = cand > S.lo_o && cand < S.hi_o && S.nnewt < 6;
    nxt = cand;
  }
  if (ok) {
    S.gallop = 0; S.nnewt++;
  } else {
    S.nnewt = 0;
    const float width = S.hi_o - S.lo_o;
    if (have && !S.edge_tried && (cand <= S.lo_o || cand >= S.hi_o)) {
      // The piece's root lies at the end of the bracket or a hair beyond it: the true root is
      // closer to that end than the offset resolves (a key whose rho is 1 - 1e-9).  Look just inside.
      const float near = fmaxf(tol, width * (1.0f / 64.0f));
      float e = NAN;
      if (cand <= S.lo_o && S.lo_o - cand <= near) e = S.lo_o + tol;
      else if (cand >= S.hi_o && cand - S.hi_o <= near) e = S.hi_o - tol;
      if (e > S.lo_o && e < S.hi_o) { nxt = e; ok = true; S.edge_tried = true; }
    }
    if (!ok && width > 2.0f * wid && S.gallop < 8) {
      const float step = ldexpf(wid, S.gallop);
      S.gallop++;
      const float c2 = fpos ? S.off + step : S.off - step;
      ok = c2 > S.lo_o && c2 < S.hi_o;
      nxt = c2;
    }
    if (!ok) {
      S.edge_tried = false;
      nxt = 0.5f * (S.lo_o + S.hi_o);
      if (!(width <= 4096.0f * wid)) {         // many binades (or not finite): halve the ordered integer keys
        const uint32_t kl = f2key(S.lo_a), kh = f2key(S.hi_a);
        if (kh > kl) {
          const float c2 = key2f(kl + (kh - kl) / 2) - S.piv;
          if (c2 > S.lo_o && c2 < S.hi_o) nxt = c2;
        }
      }
    }
  }
  if (nxt == S.off || !(nxt > S.lo_o && nxt < S.hi_o)) {   // bracket exhausted at the resolution of the offset
    S.done = true; S.a0 = ct; S.b0 = ct + cm;
    return;
  }
  if (fabsf(nxt) > 8.0f * wid) {               // keep the offset small against the keys it is subtracted from
    const float np = S.piv + nxt;
    if (np != S.piv) {
      const float delta = np - S.piv;
      S.lo_o -= delta; S.hi_o -= delta; nxt -= delta;
      S.piv = np; S.repiv = true;
    }
  }
  S.off = nxt;
}

// G lanes per row, E keys per lane (E / 4 a power of two).  KSEL: 0 = moment start, 1 / 2 = k is 1 / 2.
template <int G, int E, bool Q4, int KSEL>
__global__ void __launch_bounds__(kNtThreads, (E >= 128 ? 2 : (E >= 32 ? 4 : 6))) tk_newton_kernel(const Problem P, const float zq) {
  extern __shared__ float4 nt_smem4[];
  constexpr int R = 32 / G;                    // rows per warp
  constexpr int RS = G * E;                    // row stride in the tile
  constexpr int CH = E / 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* tile = reinterpret_cast<float*>(nt_smem4) + warp * (32 * E);
  const long long row0 = ((long long)blockIdx.x * kNtWarps + warp) * R;
  if (row0 >= P.rows) return;                  // the whole warp
  const int n = P.n, k = P.k;
  const int rl = lane / G, lig = lane % G;
  const long long row = row0 + rl;
  const bool row_ok = row < P.rows;
  const int rows_here = (int)(P.rows - row0 < (long long)R ? P.rows - row0 : (long long)R);
  const float lam = P.lam, inv_lam = P.inv_lam, lam3 = P.lam3, wid = P.lam;
  const float tol = (Q4 ? 3e-7f : 1e-6f) * wid;

  // ---- stage the warp's rows in the tile
  {
    const float* src = P.theta + row0 * (long long)n;
    if (n == RS) {
      const int total = rows_here * n;
      if (P.vec4) {
        const float4* s4 = reinterpret_cast<const float4*>(src);
        float4* t4 = reinterpret_cast<float4*>(tile);
        for (int v = lane; 4 * v < total; v += 32) t4[v] = __ldg(s4 + v);
      } else {
        for (int i = lane; i < total; i += 32) tile[i] = __ldg(src + i);
      }
    } else {
      for (int r = 0; r < rows_here; ++r) {
        if (P.vec4) {
          const float4* s4 = reinterpret_cast<const float4*>(src + (long long)r * n);
          float4* t4 = reinterpret_cast<float4*>(tile + r * RS);
          for (int v = lane; 4 * v < n; v += 32) t4[v] = __ldg(s4 + v);
        } else {
          for (int i = lane; i < n; i += 32) tile[r * RS + i] = __ldg(src + (long long)r * n + i);
        }
      }
    }
  }
  __syncwarp();

  const int rot = nt_rot<E>(lane);
  float4* span4 = reinterpret_cast<float4*>(tile + lane * E);   // this lane's E keys of its row
  const int span_n = n - lig * E;              // keys of the span that exist (may be <= 0 or >= E)
  float d[E];
  float fin = 0.0f;                            // becomes NaN when the row holds a NaN or an infinity
  {
    const bool full = row_ok && n == RS;       // every slot of the span is a key of the row
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const int cc = (c + rot) & (CH - 1);
      const float4 v = span4[cc];
      const float x4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool in = full || (row_ok && 4 * cc + j < span_n);
        d[4 * c + j] = in ? x4[j] : -INFINITY;  // slots past the end of the row never take part
        fin = fmaf(in ? x4[j] : 0.0f, 0.0f, fin);
      }
    }
  }

  // ---- start: bracket and first tau
  NtRow S;
  S.done = !row_ok; S.noblock = false; S.repiv = false;
  S.a0 = k; S.b0 = k; S.gallop = 0; S.nnewt = 0; S.prev_ct = -1; S.prev_cm = -1; S.edge_tried = false;
  S.off = 0.0f;
  float lo, hi;
  if (KSEL == 0) {
    const float x0 = tile[rl * RS];            // sums are taken about the row's first key
    float sm = 0.f, ss = 0.f, mx = -INFINITY, mn = INFINITY;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const bool in = !(d[i] == -INFINITY);
      const float dd = in ? d[i] - x0 : 0.0f;
      sm += dd; ss = fmaf(dd, dd, ss);
      mx = fmaxf(mx, d[i]);
      mn = fminf(mn, in ? d[i] : INFINITY);
    }
    sm = nt_gsum<G>(sm); ss = nt_gsum<G>(ss); mx = nt_gmax<G>(mx); mn = nt_gmin<G>(mn);
    const float inv_n = 1.0f / (float)n;
    const float mean_d = sm * inv_n;
    const float sd = sqrtf(fmaxf(ss * inv_n - mean_d * mean_d, 0.0f));
    lo = mn - wid; hi = mx;
    if (k == n) {                              // everything is selected
      S.piv = mn; S.off = -wid; S.done = true; S.noblock = true;
    } else {
      float tau0 = (x0 + mean_d) + zq * sd - (Q4 ? 0.75f : 0.5f) * lam;
      if (!(tau0 > lo && tau0 < hi)) tau0 = 0.5f * (lo + hi);
      S.piv = tau0;
    }
  } else {
    float m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int i = 0; i < E; ++i) nt_top3(d[i], m1, m2, m3);
#pragma unroll
    for (int o = G >> 1; o > 0; o >>= 1) {
      const float p1 = __shfl_xor_sync(0xffffffffu, m1, o), p2 = __shfl_xor_sync(0xffffffffu, m2, o),
                  p3 = __shfl_xor_sync(0xffffffffu, m3, o);
      nt_top3(p1, m1, m2, m3); nt_top3(p2, m1, m2, m3); nt_top3(p3, m1, m2, m3);
    }
    const float c = KSEL == 1 ? m1 : m2, sk = KSEL == 1 ? m2 : m3;   // k-th and (k+1)-th largest key
    lo = c - wid; hi = sk;
    if (!(lo < sk)) {                          // vtop(s_k) >= s_{k+1}: no violation, no block
      S.piv = c; S.off = -wid; S.done = true; S.noblock = true;
    } else {
      S.piv = 0.5f * (lo + hi);
    }
  }
  fin = nt_gsum<G>(fin);
  const bool bad = row_ok && fin != fin;
  if (!row_ok) { S.piv = 0.0f; lo = 0.0f; hi = 0.0f; }
  const bool early = S.done && S.noblock;      // pivot already exact
  S.lo_a = lo; S.hi_a = hi; S.lo_o = lo - S.piv; S.hi_o = hi - S.piv;
#pragma unroll
  for (int i = 0; i < E; ++i) d[i] -= S.piv;

  // ---- the iteration
  int passes = 0;
#pragma unroll 1
  for (; passes < kNtMaxPasses; ++passes) {
    if (__all_sync(0xffffffffu, S.done)) break;
    int ct0 = 0, ct1 = 0, cm0 = 0, cm1 = 0;
    float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, e0 = 0.f, e1 = 0.f;
    const float off = S.off;
#pragma unroll
    for (int i = 0; i < E; i += 2) {
      {
        const float t = d[i] - off;
        const bool top = t >= wid, mid = t > 0.0f && !top;
        ct0 += top; cm0 += mid;
        const float tm = mid ? t : 0.0f;
        a0 += tm;
        if (Q4) { const float t2 = tm * tm; b0 += t2; e0 = fmaf(t2, tm, e0); }
      }
      {
        const float t = d[i + 1] - off;
        const bool top = t >= wid, mid = t > 0.0f && !top;
        ct1 += top; cm1 += mid;
        const float tm = mid ? t : 0.0f;
        a1 += tm;
        if (Q4) { const float t2 = tm * tm; b1 += t2; e1 = fmaf(t2, tm, e1); }
      }
    }
    const int packed = nt_gsum<G>((ct0 + ct1) | ((cm0 + cm1) << 16));
    const float s1 = nt_gsum<G>(a0 + a1);
    float s2 = 0.f, s3 = 0.f;
    if (Q4) { s2 = nt_gsum<G>(b0 + b1); s3 = nt_gsum<G>(e0 + e1); }
    if (!S.done) {
      nt_step<Q4>(S, packed & 0xffff, packed >> 16, s1, s2, s3, k, lam, lam3, tol);
      if (S.repiv) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const int cc = (c + rot) & (CH - 1);
          const float4 v = span4[cc];
          // slots past the row stay at -infinity
          d[4 * c] = (d[4 * c] > -INFINITY) ? v.x - S.piv : d[4 * c];
          d[4 * c + 1] = (d[4 * c + 1] > -INFINITY) ? v.y - S.piv : d[4 * c + 1];
          d[4 * c + 2] = (d[4 * c + 2] > -INFINITY) ? v.z - S.piv : d[4 * c + 2];
          d[4 * c + 3] = (d[4 * c + 3] > -INFINITY) ? v.w - S.piv : d[4 * c + 3];
        }
      }
    }
  }
  int flags = 0;
  if (!S.done) {                               // cap reached: keep the last point, say so
    flags |= TK_FLAG_NOT_CONVERGED;
    S.a0 = k; S.b0 = k;
  }
  if (S.b0 <= S.a0) { S.a0 = k; S.b0 = k; }
  const bool block = S.b0 > S.a0;

  // ---- row state.  Without a block the VJP classifies by key >= pivot: any value above the
  // (k+1)-th largest key and not above the k-th serves; tau + lambda/2 is one when lambda is
  // resolved at the keys' magnitude, else the smallest capped key is looked up.
  float piv_state = S.piv, off_state = S.off;
  {
    const bool want_p = row_ok && !block && !early;
    const bool safe = wid > 9.6e-7f * (fabsf(S.piv) + fabsf(S.off));
    const bool scan = want_p && !safe;
    if (__any_sync(0xffffffffu, scan)) {
      float cmin = INFINITY;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        const int cc = (c + rot) & (CH - 1);
        const float4 v = span4[cc];
        if (d[4 * c] - S.off >= wid) cmin = fminf(cmin, v.x);
        if (d[4 * c + 1] - S.off >= wid) cmin = fminf(cmin, v.y);
        if (d[4 * c + 2] - S.off >= wid) cmin = fminf(cmin, v.z);
        if (d[4 * c + 3] - S.off >= wid) cmin = fminf(cmin, v.w);
      }
      cmin = nt_gmin<G>(cmin);
      if (scan) piv_state = cmin;
    }
    if (want_p && safe) piv_state = (S.piv + S.off) + 0.5f * wid;
    if (!block) off_state = 0.0f;
  }
  if (P.state_out && row_ok && lig == 0) {
    tk_rowstate st;
    st.pivot = piv_state; st.offset = off_state; st.a = S.a0; st.b = S.b0;
    P.state_out[row] = st;
  }

  // ---- dual map, back through the tile
  {
    const float off = S.off;
    const bool times_x = P.mode == TK_TOPK;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const int cc = (c + rot) & (CH - 1);
      float y[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a = __saturatef((d[4 * c + j] - off) * inv_lam);
        y[j] = Q4 ? a * a * a : a;
      }
      if (times_x) {
        const float4 v = span4[cc];
        y[0] *= v.x; y[1] *= v.y; y[2] *= v.z; y[3] *= v.w;
      }
      span4[cc] = make_float4(y[0], y[1], y[2], y[3]);
    }
  }
  __syncwarp();
  {
    float* dst = P.out + row0 * (long long)n;
    if (n == RS) {
      const int total = rows_here * n;
      if (P.vec4) {
        float4* d4 = reinterpret_cast<float4*>(dst);
        const float4* t4 = reinterpret_cast<const float4*>(tile);
        for (int v = lane; 4 * v < total; v += 32) d4[v] = t4[v];
      } else {
        for (int i = lane; i < total; i += 32) dst[i] = tile[i];
      }
    } else {
      for (int r = 0; r < rows_here; ++r) {
        if (P.vec4) {
          float4* d4 = reinterpret_cast<float4*>(dst + (long long)r * n);
          const float4* t4 = reinterpret_cast<const float4*>(tile + r * RS);
          for (int v = lane; 4 * v < n; v += 32) d4[v] = t4[v];
        } else {
          for (int i = lane; i < n; i += 32) dst[(long long)r * n + i] = tile[r * RS + i];
        }
      }
    }
  }
  if (P.status) {
    if (bad) flags |= TK_FLAG_NONFINITE;
    if (flags && lig == 0) atomicOr(P.status, flags);
  }
}

// z with P(N(0,1) > z) = tail, by bisection on erfc (a starting guess for the iteration: 1e-6 is plenty)
float upper_normal_quantile(double tail) {
  double lo = -8.0, hi = 8.0;
  for (int i = 0; i < 28; ++i) {
    const double mid = 0.5 * (lo + hi);
    if (0.5 * erfc(mid * 0.70710678118654752440) > tail) lo = mid; else hi = mid;
  }
  return (float)(0.5 * (lo + hi));
}

template <int G, int E, bool Q4, int KSEL>
cudaError_t nt_launch(const Problem& P, float zq, cudaStream_t stream) {
  constexpr int smem = kNtWarps * 32 * E * (int)sizeof(float);
  auto kern = tk_newton_kernel<G, E, Q4, KSEL>;
  if (smem > 48 * 1024) {
    static bool configured[64];
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (err != cudaSuccess) return err;
      if (dev >= 0 && dev < 64) configured[dev] = true;
    }
  }
  constexpr long long rows_per_block = (long long)kNtWarps * (32 / G);
  const unsigned blocks = (unsigned)((P.rows + rows_per_block - 1) / rows_per_block);
  kern<<<blocks, kNtThreads, smem, stream>>>(P, zq);
  return cudaGetLastError();
}

template <int G, int E, bool KS>
cudaError_t nt_launch_q(const Problem& P, float zq, cudaStream_t stream) {
  const bool q4 = P.q4 != 0;
  if (KS && P.k == 1) return q4 ? nt_launch<G, E, true, 1>(P, zq, stream) : nt_launch<G, E, false, 1>(P, zq, stream);
  if (KS && P.k == 2) return q4 ? nt_launch<G, E, true, 2>(P, zq, stream) : nt_launch<G, E, false, 2>(P, zq, stream);
  return q4 ? nt_launch<G, E, true, 0>(P, zq, stream) : nt_launch<G, E, false, 0>(P, zq, stream);
}

}  // namespace

int newton_max_n() { return 4096; }

// Forward pass of TK_MASK / TK_TOPK with p = 2 or 4/3, rows of up to newton_max_n() elements,
// no permutation output.
cudaError_t launch_newton(const Problem& P, cudaStream_t stream) {
  const int n = P.n;
  const float zq = upper_normal_quantile(((double)P.k - 0.5) / (double)n);
  if (n <= 8) return nt_launch_q<1, 8, true>(P, zq, stream);
  if (n <= 16) return nt_launch_q<1, 16, true>(P, zq, stream);
  if (n <= 32) return nt_launch_q<1, 32, true>(P, zq, stream);
  if (n <= 64) return nt_launch_q<1, 64, true>(P, zq, stream);
  if (n <= 128) return nt_launch_q<2, 64, true>(P, zq, stream);
  if (n <= 256) return nt_launch_q<4, 64, true>(P, zq, stream);
  if (n <= 512) return nt_launch_q<8, 64, false>(P, zq, stream);
  if (n <= 1024) return nt_launch_q<16, 64, false>(P, zq, stream);
  if (n <= 2048) return nt_launch_q<32, 64, false>(P, zq, stream);
  return nt_launch_q<32, 128, false>(P, zq, stream);
}

}  // namespace tk
