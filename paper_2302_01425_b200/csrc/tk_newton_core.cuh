// tk_newton_core.cuh -- the scalar side of the sort-free forward pass: what to do with the counts
// and power sums of one classification pass.
//
// With w = 1_k the relaxed operator's threshold tau = gamma (value of the single pooled block pool-
// adjacent-violators ends with, Sec. 5) is the root of the non-increasing function
//   F(tau) = #{key_i >= tau + width(tau)} + sum_{tau < key_i < tau + width} rho(key_i - tau) / phi'(tau) - k,
// width(tau) the key distance at which rho reaches phi'(tau): lambda for phi(x) = x (the mask: F is
// the capped-simplex condition sum y = k of Sec. 3), lambda tau^(1/(q-1)) for phi(x) = x^2/2.  On one
// piece F is the stationarity equation of that piece's candidate block, solved from the piece's
// power sums; the iteration is Newton's on the pieces, inside a bracket that every evaluated
// point tightens:
//   - a step that leaves the bracket is replaced by a step of doubling length towards the root,
//     then by bisection (of the ordered integer keys when the bracket spans many binades), and
//     after six Newton steps in a row one such step is forced: the loop ends;
//   - the root is accepted when a point reproduces the set of the pass before it and already
//     solves it to rounding, or when cm |du| is rounding-sized (F has slope >= 1/lambda until
//     it reaches an integer, so the root is then within that distance).
// tau is kept as pivot + offset and keys as d = key - pivot, so that t = d - offset is formed
// without cancellation; the row state stores exactly the pair the last pass classified with,
// and its counts, so the VJP from state sees the same classes.
#pragma once

#include <float.h>
#include <math.h>

#include "tk_common.cuh"

namespace tk {

namespace {

constexpr int kNtMaxPasses = 200;

// Root of g(u) = sum_i (t_i - u)^3 - rhs - lin u (rhs >= 0, lin >= 0) over the cm inside keys, from
// their power sums; lin = 0 for phi(x) = x, lambda^3 m for phi even, where the right-hand side
// lambda^3 m (gamma + u) moves with the root (App. A.6).  g is decreasing.  The anchor of the sums
// is the current iterate, so once the outer iteration is close the root is near 0 and Newton from
// 0 takes two steps; fp32 is enough there (u -> 0).  When the first step is not small against the
// spread of the t_i, the start is mu - cbrt(rhs / cm) instead, mu the mean of the t_i: by Jensen
// sum (t_i - u)^3 >= rhs there, which for lin = 0 puts it left of the root, where g is convex and
// Newton increases monotonically to the root.  c0 = g(0).
__device__ __forceinline__ float nt_cubic(int cm, float s1, float s2, float s3, float rhs, float lin, float c0) {
  const float fcm = (float)cm;
  const float inv_cm = __fdividef(1.0f, fcm);
  const float spread2 = s2 * inv_cm;                       // mean of t^2
  float u = __fdividef(c0, 3.0f * s2 + lin);               // Newton step from 0
  if (u * u > 0.01f * spread2) u = s1 * inv_cm - cbrtf(rhs * inv_cm);
  const float spread = sqrtf(spread2);
#pragma unroll 1
  for (int it = 0; it < 8; ++it) {
    const float g = ((-fcm * u + 3.0f * s1) * u - (3.0f * s2 + lin)) * u + c0;
    const float gp = -3.0f * ((fcm * u - 2.0f * s1) * u + s2) - lin;
    if (!(gp < 0.0f)) break;
    const float st = -__fdividef(g, gp);
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

// The next offset when the piece's own solution cannot be taken as it is: it left the bracket, there was
// no piece to solve, six Newton steps have gone by, or the offset has grown large against lambda.  Out
// of line: the common pass never comes here, and its code stays short.
static __device__ __noinline__ NtRow nt_step_slow(NtRow S, int ct, int cm, int m, float du, bool have,
                                                  bool fpos, float wid, float tol, bool nudge, bool mag) {
  bool ok = false;
  float nxt = S.off;
  float cand = S.off;
  if (have) {
    cand = S.off + du;
    // every inside key would have to reach the cap: aim just past it, so that they read as capped
    if (nudge) cand -= 0.5f * tol;
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
    return S;
  }
  // keep the offset small against the keys it is subtracted from; phi even: and against tau itself,
  // which the width and the piece's equation depend on (tau = pivot + offset must not cancel)
  if (fabsf(nxt) > 8.0f * wid || (mag && S.piv + nxt < 0.5f * S.piv)) {
    const float np = S.piv + nxt;
    if (np != S.piv) {
      const float delta = np - S.piv;
      S.lo_o -= delta; S.hi_o -= delta; nxt -= delta;
      S.piv = np; S.repiv = true;
    }
  }
  S.off = nxt;
  return S;
}

// Key distance above tau at which an inside key reaches the cap: rho(width) = phi'(tau).
template <bool Q4, bool MAG>
__device__ __forceinline__ float nt_width(float tau, float lam) {
  if (!MAG) return lam;
  const float t = fmaxf(tau, 0.0f);
  return Q4 ? lam * cbrtf(t) : lam * t;
}

// What one pass found at S.off (classes against width wid, sums of t, t^2, t^3 over the inside keys)
// -> the next offset, or the end of the iteration.  The piece's equation (Sec. 5 example, App. A.6):
//   phi = x,    q = 2:  sum (t_i - u) = lambda m                       q = 4:  sum (t_i - u)^3 = lambda^3 m
//   phi = x^2/2, q = 2: sum (t_i - u) = lambda m (gamma + u)           q = 4:  sum (t_i - u)^3 = lambda^3 m (gamma + u)
// with gamma = pivot + offset the point of the pass and m = k - #capped.
template <bool Q4, bool MAG>
__device__ __forceinline__ void nt_step(NtRow& S, int ct, int cm, float s1, float s2, float s3, int k,
                                        float lam, float lam3, float wid, float tol) {
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
    const float gam = S.piv + S.off;
    float c0;
    if (!Q4) {
      const float lm = lam * (float)m;
      c0 = s1 - (MAG ? lm * gam : lm);
      du = __fdividef(c0, MAG ? (float)cm + lm : (float)cm);
    } else {
      const float l3m = lam3 * (float)m;
      const float rhs = MAG ? l3m * fmaxf(gam, 0.0f) : l3m;
      c0 = s3 - rhs;
      du = nt_cubic(cm, s1, s2, s3, rhs, MAG ? l3m : 0.0f, c0);
      if ((du > 0.0f) != (c0 > 0.0f)) du = __fdividef(c0, 3.0f * s2 + (MAG ? l3m : 0.0f));
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
  // the common case: the piece's solution lies inside the bracket and near the pivot
  const float cand = S.off + du;
  const bool nudge = m == cm;                  // every inside key would have to reach the cap
  if (have && !nudge && cand > S.lo_o && cand < S.hi_o && S.nnewt < 6 && fabsf(cand) <= 8.0f * wid &&
      !(MAG && S.piv + cand < 0.5f * S.piv)) {
    S.gallop = 0; S.nnewt++; S.off = cand;
    return;
  }
  S = nt_step_slow(S, ct, cm, m, du, have, fpos, wid, tol, nudge, MAG);
}

__device__ __forceinline__ void nt_row_init(NtRow& S, int k) {
  S.done = false; S.noblock = false; S.repiv = false;
  S.a0 = k; S.b0 = k; S.gallop = 0; S.nnewt = 0; S.prev_ct = -1; S.prev_cm = -1; S.edge_tried = false;
  S.off = 0.0f; S.piv = 0.0f; S.lo_o = -INFINITY; S.hi_o = INFINITY; S.lo_a = -FLT_MAX; S.hi_a = FLT_MAX;
}

}  // namespace

}  // namespace tk
