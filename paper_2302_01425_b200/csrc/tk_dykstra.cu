// tk_dykstra.cu -- the alternating-projection solver path (Algorithm 1 and
// App. A.8 of the paper) for rows held on chip, a fixed number of sweeps.
//
// After the same sort as the exact path, the isotonic problem is iterated on
// the two families of adjacent pairs C1 = {(1,2),(3,4),..}, C2 = {(2,3),(4,5),..}:
//
//  p = 2: Dykstra's projection of z onto C1 n C2 in the metric c, with
//    z_i = s_i - lambda w_i, c_i = 1          (phi = x)
//    z_i = s_i / c_i,        c_i = 1 + lambda w_i   (phi = x^2/2; completing the
//    square of h_i).  The linear term is applied once, through z (the printed
//    iteration, which subtracts w in both half-steps, converges to the
//    projection of s - 2w).  The correction kept for a pair (a, b) is one scalar
//    delta >= 0: the pair's corrections are (-c_b delta, +c_a delta).
//  p = 4/3, phi = x: block coordinate ascent on the duals alpha_j >= 0 of
//    v_j >= v_{j+1}; each coordinate solves its two-variable problem in closed
//    form (depressed cubic t^3 + 3 d^2 t + B = 0 by Cardano, one Newton step),
//    odd coordinates then even coordinates.  The output needs no cube root:
//    rho(s_i - v_i) = w_i - alpha_i + alpha_{i-1}.
//
// Each thread (lane) owns an even number of consecutive sorted ranks, so every C1
// pair is thread-local and one C2 pair per thread crosses to the next thread.
//
// Rows of 16385..131072 elements do not fit one thread block's registers: a
// thread-block cluster of up to 8 blocks shares the row, 16384 consecutive sorted
// ranks per block, and the one pair that crosses from a block to the next is
// exchanged through distributed shared memory.  The sort of such a row is the
// global-memory radix sort (tk_long.cu); the iterate never leaves the chip.
#include <cooperative_groups.h>

#include "tk_common.cuh"
#include "tk_cta_sort.cuh"
#include "tk_group_sort.cuh"

namespace tk {

namespace {

// One Dykstra step on a pair in the metric (ca, cb): a, b are the current iterate, delta the
// stored correction; on return a >= b holds and delta is the new correction.
__device__ __forceinline__ void dyk_pair(float& a, float& b, float& delta, float ca, float cb) {
  const float ta = a - cb * delta, tb = b + ca * delta;
  const float d = fmaxf(0.0f, (tb - ta) / (ca + cb));
  a = ta + cb * d;
  b = tb - ca * d;
  delta = d;
}

// Dual coordinate of the constraint between keys s1 >= s2 (weights w1, w2), neighbours' duals fixed.
__device__ __forceinline__ float bca_alpha(float s1, float s2, float w1, float w2, float a_prev,
                                           float a_next, const Math& M) {
  const float c1 = w1 + a_prev, c2 = w2 - a_next;
  // s1 >= s2, so the separate minimisers s_i - lam cbrt(c_i) are in order whenever c1 <= c2: most
  // pairs (equal weights, no active neighbour) end here without a cube root
  if (c1 <= c2) return 0.0f;
  const float v1 = s1 - M.lam * cbrtf(c1), v2 = s2 - M.lam * cbrtf(c2);
  if (v1 >= v2) return 0.0f;
  const float d = 0.5f * (s1 - s2), m = 0.5f * (s1 + s2);
  const float B = 0.5f * M.lam3 * (c1 + c2);
  const float d2 = d * d;
  const float R = sqrtf(0.25f * B * B + d2 * d2 * d2);
  const float big = -copysignf(cbrtf(0.5f * fabsf(B) + R), B);
  float t = (big != 0.0f) ? big - d2 / big : 0.0f;
  {   // one Newton step on the increasing cubic t^3 + 3 d^2 t + B
    const float f = fmaf(t * t + 3.0f * d2, t, B), fp = 3.0f * (t * t + d2);
    if (fp > 0.0f) t -= f / fp;
  }
  const float z = (s1 - (m + t)) * M.inv_lam;
  return fmaxf(0.0f, c1 - z * z * z);
}

// ---- the same coordinate step for any q and for phi even (App. A.8 leaves the two-variable problem to a
// root solver; the closed form above is the special case q = 4, phi = x).  rho is odd: sign(t) |t/lambda|^(q-1).
__device__ __forceinline__ float bca_rho(const Math& M, float t) {
  const float a = fabsf(t) * M.inv_lam;
  return copysignf(M.gen ? powf(a, M.qm1) : (M.q4 ? a * a * a : a), t);
}
__device__ __forceinline__ float bca_drho(const Math& M, float t) {
  const float a = fabsf(t) * M.inv_lam;
  return (M.gen ? M.qm1 * powf(a, M.qm1 - 1.0f) : (M.q4 ? 3.0f * a * a : 1.0f)) * M.inv_lam;
}
__device__ __forceinline__ float bca_rho_inv(const Math& M, float z) {
  const float a = fabsf(z);
  return copysignf(M.lam * (M.gen ? powf(a, 1.0f / M.qm1) : (M.q4 ? cbrtf(a) : a)), z);
}
// Root of an increasing function inside [lo, hi] (f(lo) <= 0 <= f(hi)): Newton, bisection when a step
// leaves the bracket.  fd(x, f, df) evaluates the function and its derivative.
template <class FD>
__device__ __forceinline__ float bca_root(float lo, float hi, float x, FD fd) {
#pragma unroll 1
  for (int it = 0; it < 60; ++it) {
    float f, df;
    fd(x, f, df);
    if (f > 0.0f) hi = x; else lo = x;
    float nx = df > 0.0f ? x - f / df : 0.5f * (lo + hi);
    if (!(nx > lo && nx < hi)) nx = 0.5f * (lo + hi);
    if (fabsf(nx - x) <= 1e-7f * fabsf(nx) + 1e-30f || !(hi > lo)) { x = nx; break; }
    x = nx;
  }
  return x;
}
// argmin_v r*(s - v) + w phi(v) + c v: -rho(s - v) + w phi'(v) + c = 0
__device__ __forceinline__ float bca_shifted(const Math& M, float s, float w, float c) {
  if (!M.mag || w == 0.0f) return s - bca_rho_inv(M, (M.mag ? 0.0f : w) + c);
  // phi even, w = 1: with t = s - v, rho(t) + t = s + c, t between 0 and s + c
  const float R = s + c;
  if (R == 0.0f) return s;
  const float lo = fminf(0.0f, R), hi = fmaxf(0.0f, R);
  const float t = bca_root(lo, hi, 0.5f * R, [&](float x, float& f, float& df) {
    f = bca_rho(M, x) + x - R; df = bca_drho(M, x) + 1.0f; });
  return s - t;
}
// the dual of the constraint between keys s1 >= s2, neighbours' duals fixed
__device__ __forceinline__ float bca_alpha_any(float s1, float s2, float w1, float w2, float a_prev, float a_next,
                                              const Math& M) {
  const float c1 = a_prev, c2 = -a_next;
  if (!M.mag && w1 + c1 <= w2 + c2) return 0.0f;           // separate minimisers in order (rho_inv is increasing)
  const float v1 = bca_shifted(M, s1, w1, c1), v2 = bca_shifted(M, s2, w2, c2);
  if (v1 >= v2) return 0.0f;
  const float ws = w1 + w2, cs = c1 + c2;
  const float g = bca_root(v1, v2, 0.5f * (v1 + v2), [&](float x, float& f, float& df) {
    f = -bca_rho(M, s1 - x) - bca_rho(M, s2 - x) + (M.mag ? ws * x : ws) + cs;
    df = bca_drho(M, s1 - x) + bca_drho(M, s2 - x) + (M.mag ? ws : 0.0f); });
  return fmaxf(0.0f, -bca_rho(M, s1 - g) + (M.mag ? w1 * g : w1) + a_prev);
}
// y_i = rho(s_i - v_i) at the primal iterate v_i = argmin h_i(v) + (alpha_{i-1} - alpha_i) v
__device__ __forceinline__ float bca_output(const Math& M, float s, float w, float a_im1, float a_i) {
  if (!M.mag) return w + a_im1 - a_i;
  const float v = fmaxf(bca_shifted(M, s, w, a_im1 - a_i), 0.0f);
  return bca_rho(M, s - v);
}

// The solver on E consecutive ranks per thread.  Exchange with the neighbouring threads goes
// through the two callables: next0(x) returns the NEXT thread's x, prev_last(x) the PREVIOUS thread's.
// On return y[i] = rho(s_i - v_i).
// MAG (phi even) is a template flag: for phi = x every metric weight is the constant 1, the pair
// projection loses its division and the weights their registers.
// key_again(i): the key s[i] once more, for the output map of the p = 2 iteration, which does not
// touch s between its first line and its last: a kernel short of registers reads it from memory there.
// TOL (run to a tolerance, tk_opts.tol > 0): the largest move of an entry of the iterate (p = 2) or of a
// dual (p = 4/3) in any projection of a sweep is taken over the row by row_max(x), which returns the same
// value to every thread of the row; the sweeps end when it is at most P.tol, or at the cap `sweeps`
// (returns false then: not converged).
template <int E, bool MAG, bool TOL, typename NextF, typename PrevF, typename SyncF, typename KeyF, typename MaxF>
__device__ __forceinline__ bool solve_pairs_m(const Problem& P, const Math& M, const float (&s)[E], int rank0,
                                            bool has_next, bool has_prev, NextF next_of, PrevF prev_of,
                                            SyncF sync, KeyF key_again, MaxF row_max, float (&y)[E]) {
  const int n = P.n, k = P.k;
  const int sweeps = P.sweeps > 0 ? P.sweeps : 100;
  bool met = !TOL;
  const float s_next = next_of(s[0]);                      // key of the next thread's first rank
  sync();
  const bool cross = has_next && (rank0 + E) < n;          // pair (rank0 + E - 1, rank0 + E) exists
  auto wgt = [&](int rk) -> float { return rk < k ? 1.0f : 0.0f; };
  if (!M.q4) {
    float v[E], c[E], pd[E / 2], qd[E / 2];
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float w = wgt(rank0 + i);
      c[i] = MAG ? 1.0f + M.lam * w : 1.0f;
      v[i] = MAG ? s[i] / c[i] : s[i] - M.lam * w;
    }
#pragma unroll
    for (int j = 0; j < E / 2; ++j) { pd[j] = 0.0f; qd[j] = 0.0f; }
    const float c_next = MAG ? 1.0f + M.lam * wgt(rank0 + E) : 1.0f;
#pragma unroll 1
    for (int it = 0; it < sweeps; ++it) {
      float chg = 0.0f;                                    // TOL: largest move of one of this thread's entries
#pragma unroll
      for (int j = 0; j < E / 2; ++j)
        if (rank0 + 2 * j + 1 < n) {
          const float o0 = v[2 * j], o1 = v[2 * j + 1];
          dyk_pair(v[2 * j], v[2 * j + 1], pd[j], c[2 * j], c[2 * j + 1]);
          if (TOL) chg = fmaxf(chg, fmaxf(fabsf(v[2 * j] - o0), fabsf(v[2 * j + 1] - o1)));
        }
      // C2: the pair that crosses to the next thread, then the thread-local ones
      float nb = next_of(v[0]);
      float mine = v[E - 1];
      if (cross) {
        const float o0 = mine, o1 = nb;
        dyk_pair(mine, nb, qd[E / 2 - 1], c[E - 1], c_next);
        if (TOL) chg = fmaxf(chg, fmaxf(fabsf(mine - o0), fabsf(nb - o1)));
      }
      v[E - 1] = mine;
#pragma unroll
      for (int j = 0; j < E / 2 - 1; ++j)
        if (rank0 + 2 * j + 2 < n) {
          const float o0 = v[2 * j + 1], o1 = v[2 * j + 2];
          dyk_pair(v[2 * j + 1], v[2 * j + 2], qd[j], c[2 * j + 1], c[2 * j + 2]);
          if (TOL) chg = fmaxf(chg, fmaxf(fabsf(v[2 * j + 1] - o0), fabsf(v[2 * j + 2] - o1)));
        }
      sync();
      const float back = prev_of(nb);                      // what the previous thread made of my first rank
      if (has_prev && rank0 < n) v[0] = back;
      sync();
      if (TOL && row_max(chg) <= P.tol) { met = true; break; }
    }
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float vi = MAG ? fmaxf(v[i], 0.0f) : v[i];
      y[i] = (key_again(i) - vi) * M.inv_lam;
    }
  } else {
    // alpha of constraint (rank0 + i, rank0 + i + 1): i even -> ao[i/2], i odd -> ae[i/2]
    float ao[E / 2], ae[E / 2];
#pragma unroll
    for (int j = 0; j < E / 2; ++j) { ao[j] = 0.0f; ae[j] = 0.0f; }
    float prev_e = 0.0f;                                   // previous thread's last even-family dual
#pragma unroll 1
    for (int it = 0; it < sweeps; ++it) {
      float chg = 0.0f;                                    // TOL: largest move of one of this thread's duals
#pragma unroll
      for (int j = 0; j < E / 2; ++j) {
        const int rk = rank0 + 2 * j;
        if (rk + 1 < n) {
          const float a_prev = (j == 0) ? prev_e : ae[j - 1];
          const float old = ao[j];
          ao[j] = bca_alpha(s[2 * j], s[2 * j + 1], wgt(rk), wgt(rk + 1), a_prev, ae[j], M);
          if (TOL) chg = fmaxf(chg, fabsf(ao[j] - old));
        }
      }
      const float next_o = next_of(ao[0]);
      sync();
#pragma unroll
      for (int j = 0; j < E / 2; ++j) {
        const int rk = rank0 + 2 * j + 1;
        const float old = ae[j];
        if (j < E / 2 - 1) {
          if (rk + 1 < n) ae[j] = bca_alpha(s[2 * j + 1], s[2 * j + 2], wgt(rk), wgt(rk + 1), ao[j], ao[j + 1], M);
        } else if (cross) {
          const float a_next = (rk + 2 < n) ? next_o : 0.0f;
          ae[j] = bca_alpha(s[E - 1], s_next, wgt(rk), wgt(rk + 1), ao[j], a_next, M);
        }
        if (TOL) chg = fmaxf(chg, fabsf(ae[j] - old));
      }
      const float pe = prev_of(ae[E / 2 - 1]);
      prev_e = has_prev ? pe : 0.0f;
      sync();
      if (TOL && row_max(chg) <= P.tol) { met = true; break; }
    }
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float a_i = (i & 1) ? ae[i / 2] : ao[i / 2];
      const float a_im1 = (i == 0) ? prev_e : ((i & 1) ? ao[i / 2] : ae[i / 2 - 1]);
      y[i] = wgt(rank0 + i) - a_i + a_im1;
    }
  }
  return met;
}

// returns false when a run to tolerance (TOL) stopped at the cap
template <int E, bool TOL, typename NextF, typename PrevF, typename SyncF, typename KeyF, typename MaxF>
__device__ __forceinline__ bool solve_pairs(const Problem& P, const Math& M, const float (&s)[E], int rank0,
                                            bool has_next, bool has_prev, NextF next_of, PrevF prev_of,
                                            SyncF sync, KeyF key_again, MaxF row_max, float (&y)[E]) {
  if (M.mag) return solve_pairs_m<E, true, TOL>(P, M, s, rank0, has_next, has_prev, next_of, prev_of, sync, key_again, row_max, y);
  return solve_pairs_m<E, false, TOL>(P, M, s, rank0, has_next, has_prev, next_of, prev_of, sync, key_again, row_max, y);
}

// ------------------------------------------------------------------ rows of up to 256 elements
template <int G>
__global__ void __launch_bounds__(128) tk_group_dykstra_kernel(const Problem P) {
  constexpr int N = G * EPL;
  constexpr int GROUPS = 128 / G;
  constexpr int STRIDE = N + (N >> 3) + 1;
  __shared__ float stage_all[GROUPS][STRIDE];
  const int tid = threadIdx.x;
  const int grp = tid / G, lig = tid % G;
  const long long row = (long long)blockIdx.x * GROUPS + grp;
  if (row >= P.rows) return;
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << ((tid & 31) / G * G);
  const int n = P.n;
  const Math M = make_math_q24(P);
  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[EPL];
  bool bad = false;
  group_load_pack(P, x_row, lig, M.mag, r, bad);
  group_sort<G>(r, lig, mask);
  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
#pragma unroll
    for (int i = 0; i < EPL; ++i) if (EPL * lig + i < n) pr[EPL * lig + i] = un_idx(r[i]);
  }
  float s[EPL], y[EPL];
#pragma unroll
  for (int i = 0; i < EPL; ++i) s[i] = un_key(r[i]);
  auto next_of = [&](float x) -> float { return __shfl_down_sync(mask, x, 1, G); };
  auto prev_of = [&](float x) -> float { return __shfl_up_sync(mask, x, 1, G); };
  auto sync = [&]() {};
  auto row_max = [&](float x) -> float {
#pragma unroll
    for (int o = G >> 1; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(mask, x, o, G));
    return x;
  };
  auto key_of = [&](int i) -> float { return s[i]; };
  const bool met = P.tol > 0.0f
      ? solve_pairs<EPL, true>(P, M, s, EPL * lig, lig < G - 1, lig > 0, next_of, prev_of, sync, key_of, row_max, y)
      : solve_pairs<EPL, false>(P, M, s, EPL * lig, lig < G - 1, lig > 0, next_of, prev_of, sync, key_of, row_max, y);
  if (!met && lig == 0 && P.status) atomicOr(P.status, TK_FLAG_NOT_CONVERGED);

  float* stage = stage_all[grp];
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int idx = un_idx(r[i]);
    if (EPL * lig + i < n && idx < n) stage[pad8(idx)] = (M.mag && un_neg(r[i])) ? -y[i] : y[i];
  }
  __syncwarp(mask);
  float* o_row = P.out + row * (long long)n;
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int idx = EPL * lig + i;
    if (idx < n) { float q = stage[pad8(idx)]; if (P.mode == TK_TOPK) q *= __ldg(x_row + idx); o_row[idx] = q; }
  }
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
}

// ------------------------------------------------------------------ p = 4/3, rows of up to 256 elements
// The sub-warp layout of the kernel above with the pairs dealt to the row's G lanes round-robin (lane l owns
// pairs l, l + G, ...): the pooled block is a run of consecutive ranks, so at every step of a half-sweep the
// lanes of a row are either all on heavy pairs (cube roots, Cardano) or all on light ones, where with
// consecutive ranks per lane one or two lanes of a row did all the heavy work and the warp waited for them.
// The neighbour duals cross lanes by shuffles: pair q - 1 is the lane below at the same step, or the row's
// last lane at the step before; pair q + 1 the lane above, or the row's first lane at the next step.
template <int G, bool ANY>
__global__ void __launch_bounds__(128, ANY ? 4 : 6) tk_group_bca_kernel(const Problem P) {
  constexpr int N = G * EPL;
  constexpr int GROUPS = 128 / G;
  constexpr int STRIDE = N + (N >> 3) + 1;
  constexpr int H = EPL / 2;                                // pairs per lane
  __shared__ float stage_all[GROUPS][STRIDE];
  const int tid = threadIdx.x;
  const int grp = tid / G, lig = tid % G;
  const long long row = (long long)blockIdx.x * GROUPS + grp;
  if (row >= P.rows) return;
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << ((tid & 31) / G * G);
  const int n = P.n, k = P.k;
  Math M = make_math(P);
  if (!ANY) { M.gen = false; M.mag = false; }
  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[EPL];
  bool bad = false;
  group_load_pack(P, x_row, lig, P.mode == TK_TOPKMAG, r, bad);
  group_sort<G>(r, lig, mask);
  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
#pragma unroll
    for (int i = 0; i < EPL; ++i) if (EPL * lig + i < n) pr[EPL * lig + i] = un_idx(r[i]);
  }
  float* stage = stage_all[grp];
  // the sorted keys by rank, then this lane's pairs
#pragma unroll
  for (int i = 0; i < EPL; ++i) stage[pad8(EPL * lig + i)] = un_key(r[i]);
  __syncwarp(mask);
  auto wgt = [&](int rk) -> float { return rk < k ? 1.0f : 0.0f; };
  float s_lo[H], s_hi[H], s_nx[H], ao[H], ae[H];
#pragma unroll
  for (int j = 0; j < H; ++j) {
    const int q = lig + j * G;
    s_lo[j] = stage[pad8(2 * q)];
    s_hi[j] = stage[pad8(2 * q + 1)];
    s_nx[j] = (2 * q + 2 < N) ? stage[pad8(2 * q + 2)] : 0.0f;
    ao[j] = 0.0f; ae[j] = 0.0f;
  }
  __syncwarp(mask);
  const int sweeps = P.sweeps > 0 ? P.sweeps : 100;
  const bool tol_mode = P.tol > 0.0f;
  bool met = !tol_mode;
#pragma unroll 1
  for (int it = 0; it < sweeps; ++it) {
    float chg = 0.0f;
    // odd family: constraint (2q, 2q + 1); neighbours: the even duals of pairs q - 1 and q
#pragma unroll
    for (int j = 0; j < H; ++j) {
      const int q = lig + j * G;
      const float below = __shfl_up_sync(mask, ae[j], 1, G);
      const float wrap = j > 0 ? __shfl_sync(mask, ae[j > 0 ? j - 1 : 0], G - 1, G) : 0.0f;
      const float a_prev = lig > 0 ? below : wrap;
      if (2 * q + 1 < n) {
        const float old = ao[j];
        ao[j] = ANY ? bca_alpha_any(s_lo[j], s_hi[j], wgt(2 * q), wgt(2 * q + 1), a_prev, ae[j], M)
                    : bca_alpha(s_lo[j], s_hi[j], wgt(2 * q), wgt(2 * q + 1), a_prev, ae[j], M);
        chg = fmaxf(chg, fabsf(ao[j] - old));
      }
    }
    // even family: constraint (2q + 1, 2q + 2); neighbours: the odd duals of pairs q and q + 1
#pragma unroll
    for (int j = 0; j < H; ++j) {
      const int q = lig + j * G;
      const float above = __shfl_down_sync(mask, ao[j], 1, G);
      const float wrap = j < H - 1 ? __shfl_sync(mask, ao[j < H - 1 ? j + 1 : j], 0, G) : 0.0f;
      const float a_up = lig < G - 1 ? above : wrap;
      if (2 * q + 2 < n) {
        const float a_next = (2 * q + 3 < n) ? a_up : 0.0f;
        const float old = ae[j];
        ae[j] = ANY ? bca_alpha_any(s_hi[j], s_nx[j], wgt(2 * q + 1), wgt(2 * q + 2), ao[j], a_next, M)
                    : bca_alpha(s_hi[j], s_nx[j], wgt(2 * q + 1), wgt(2 * q + 2), ao[j], a_next, M);
        chg = fmaxf(chg, fabsf(ae[j] - old));
      }
    }
    if (tol_mode) {
#pragma unroll
      for (int o = G >> 1; o > 0; o >>= 1) chg = fmaxf(chg, __shfl_xor_sync(mask, chg, o, G));
      if (chg <= P.tol) { met = true; break; }
    }
  }
  if (!met && lig == 0 && P.status) atomicOr(P.status, TK_FLAG_NOT_CONVERGED);
  // y_i = w_i - alpha_i + alpha_{i-1}, by rank into the stage, then back to the sorted registers' layout
#pragma unroll
  for (int j = 0; j < H; ++j) {
    const int q = lig + j * G;
    const float below = __shfl_up_sync(mask, ae[j], 1, G);
    const float wrap = j > 0 ? __shfl_sync(mask, ae[j > 0 ? j - 1 : 0], G - 1, G) : 0.0f;
    const float a_im1 = lig > 0 ? below : wrap;
    stage[pad8(2 * q)] = ANY ? bca_output(M, s_lo[j], wgt(2 * q), a_im1, ao[j]) : wgt(2 * q) - ao[j] + a_im1;
    stage[pad8(2 * q + 1)] = ANY ? bca_output(M, s_hi[j], wgt(2 * q + 1), ao[j], ae[j]) : wgt(2 * q + 1) - ae[j] + ao[j];
  }
  __syncwarp(mask);
  float y[EPL];
#pragma unroll
  for (int i = 0; i < EPL; ++i) y[i] = stage[pad8(EPL * lig + i)];
  __syncwarp(mask);
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int idx = un_idx(r[i]);
    if (EPL * lig + i < n && idx < n) stage[pad8(idx)] = (ANY && M.mag && un_neg(r[i])) ? -y[i] : y[i];
  }
  __syncwarp(mask);
  float* o_row = P.out + row * (long long)n;
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int idx = EPL * lig + i;
    if (idx < n) { float q = stage[pad8(idx)]; if (P.mode == TK_TOPK) q *= __ldg(x_row + idx); o_row[idx] = q; }
  }
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
}

// ------------------------------------------------------------------ rows of up to 16384 elements
template <int E, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) tk_cta_dykstra_kernel(const Problem P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int T = blockDim.x, t = threadIdx.x, n = P.n, N = P.N;
  const long long row = blockIdx.x;
  const Math M = make_math_q24(P);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  float* stage = reinterpret_cast<float*>(smem_raw);
  float* xch_a = reinterpret_cast<float*>(keys + pad(N) + 1);   // 2 x (T + 2) floats
  float* xch_b = xch_a + (T + 2);
  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[E];
  bool bad = false;
  cta_load_sort<E>(P, x_row, keys, r, bad);
  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
    for (int i = t; i < n; i += T) pr[i] = un_idx(keys[pad(i)]);
  }
  float s[E], y[E];
#pragma unroll
  for (int i = 0; i < E; ++i) s[i] = un_key(r[i]);
  // Neighbour exchange: write own value, barrier, read the neighbour's slot.  The solver alternates
  // the two kinds of exchange and each has its own array, so a slot is overwritten only after the
  // barrier of the other kind's exchange, which every thread passes after its read: the solver's
  // sync() between exchanges needs a barrier only after the one exchange that precedes the sweeps
  // (it is followed by another of its kind).  Two block barriers per sweep.
  auto next_of = [&](float x) -> float { xch_a[t] = x; __syncthreads(); return (t + 1 < T) ? xch_a[t + 1] : 0.0f; };
  auto prev_of = [&](float x) -> float { xch_b[t] = x; __syncthreads(); return (t > 0) ? xch_b[t - 1] : 0.0f; };
  bool before_sweeps = true;
  auto sync = [&]() { if (before_sweeps) { __syncthreads(); before_sweeps = false; } };
  // largest value over the block: warp maxima through a third array (its two barriers also fence the
  // exchanges of the sweep that follows against this one's)
  __shared__ float red_max[32];
  auto row_max = [&](float x) -> float {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    __syncthreads();
    if ((t & 31) == 0) red_max[t >> 5] = x;
    __syncthreads();
    float r = red_max[0];
    for (int w = 1; w < (T >> 5); ++w) r = fmaxf(r, red_max[w]);
    return r;
  };
  auto key_of = [&](int i) -> float { return s[i]; };
  const bool met = P.tol > 0.0f
      ? solve_pairs<E, true>(P, M, s, E * t, t + 1 < T, t > 0, next_of, prev_of, sync, key_of, row_max, y)
      : solve_pairs<E, false>(P, M, s, E * t, t + 1 < T, t > 0, next_of, prev_of, sync, key_of, row_max, y);
  if (!met && t == 0 && P.status) atomicOr(P.status, TK_FLAG_NOT_CONVERGED);

  __syncthreads();
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const int idx = un_idx(r[i]);
    if (t * E + i < n && idx < n) stage[idx] = (M.mag && un_neg(r[i])) ? -y[i] : y[i];
  }
  __syncthreads();
  float* o_row = P.out + row * (long long)n;
  for (int i = t; i < n; i += T) { float q = stage[i]; if (P.mode == TK_TOPK) q *= __ldg(x_row + i); o_row[i] = q; }
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
}

// ------------------------------------------------------------------ p = 4/3, rows of 257..16384 elements
// The dual block coordinate ascent of App. A.8 with the pairs dealt to the threads round-robin: thread t
// owns pairs t, t + T, t + 2T, ... (pair q = ranks 2q, 2q + 1).  The pooled block is a run of consecutive
// ranks and only its pairs pay the cube roots and the Cardano step; with consecutive ranks per thread it
// sits in a few warps that set the pace while the rest of the block waits at the sweep's barriers, dealt
// round-robin every warp holds its share.  The price: every pair's neighbour dual crosses threads, so each
// half-sweep publishes its family's duals in shared memory (one array per family, a barrier after each
// write: two barriers per sweep as before).  Pairs of one family do not touch each other, so the iterates
// are those of the kernel above and of the oracle, sweep by sweep.
// ANY: any q and phi even through the root-solving pair step (one Newton iteration inside another: slow,
// but the same sweeps); otherwise q = 4, phi = x with the closed form.
template <int E, int MAXT, int MINB, bool ANY>
__global__ void __launch_bounds__(MAXT, MINB) tk_cta_bca_kernel(const Problem P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int H = E / 2;                                  // pairs per thread
  const int T = blockDim.x, t = threadIdx.x, n = P.n, N = P.N, k = P.k;
  const long long row = blockIdx.x;
  Math M = make_math(P);
  if (!ANY) { M.gen = false; M.mag = false; }
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  float* xo = reinterpret_cast<float*>(keys + pad(N) + 1);  // odd-family duals, one per pair: N / 2 floats
  float* xe = xo + N / 2;                                   // even-family duals
  float* stage = xo;                                        // the output, by original index (N floats: both arrays)
  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[E];
  bool bad = false;
  cta_load_sort<E>(P, x_row, keys, r, bad);
  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
    for (int i = t; i < n; i += T) pr[i] = un_idx(keys[pad(i)]);
  }
  auto wgt = [&](int rk) -> float { return rk < k ? 1.0f : 0.0f; };
  // this thread's pairs: keys of ranks 2q, 2q + 1 and 2q + 2 (sorted order is in shared memory)
  float s_lo[H], s_hi[H], s_nx[H], ao[H], ae[H];
#pragma unroll
  for (int j = 0; j < H; ++j) {
    const int q = t + j * T;
    s_lo[j] = un_key(keys[pad(2 * q)]);
    s_hi[j] = un_key(keys[pad(2 * q + 1)]);
    s_nx[j] = (2 * q + 2 < N) ? un_key(keys[pad(2 * q + 2)]) : 0.0f;
    ao[j] = 0.0f; ae[j] = 0.0f;
    xe[q] = 0.0f;
  }
  __shared__ float red_max[32];
  auto row_max = [&](float x) -> float {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    __syncthreads();
    if ((t & 31) == 0) red_max[t >> 5] = x;
    __syncthreads();
    float m = red_max[0];
    for (int w = 1; w < (T >> 5); ++w) m = fmaxf(m, red_max[w]);
    return m;
  };
  const int sweeps = P.sweeps > 0 ? P.sweeps : 100;
  const bool tol_mode = P.tol > 0.0f;
  bool met = !tol_mode;
  __syncthreads();
#pragma unroll 1
  for (int it = 0; it < sweeps; ++it) {
    float chg = 0.0f;
    // odd family: constraint (2q, 2q + 1); neighbours: the even duals of pairs q - 1 and q
#pragma unroll
    for (int j = 0; j < H; ++j) {
      const int q = t + j * T;
      if (2 * q + 1 < n) {
        const float a_prev = q > 0 ? xe[q - 1] : 0.0f;
        const float old = ao[j];
        ao[j] = ANY ? bca_alpha_any(s_lo[j], s_hi[j], wgt(2 * q), wgt(2 * q + 1), a_prev, ae[j], M)
                    : bca_alpha(s_lo[j], s_hi[j], wgt(2 * q), wgt(2 * q + 1), a_prev, ae[j], M);
        chg = fmaxf(chg, fabsf(ao[j] - old));
      }
      xo[q] = ao[j];
    }
    __syncthreads();
    // even family: constraint (2q + 1, 2q + 2); neighbours: the odd duals of pairs q and q + 1
#pragma unroll
    for (int j = 0; j < H; ++j) {
      const int q = t + j * T;
      if (2 * q + 2 < n) {
        const float a_next = (2 * q + 3 < n) ? xo[q + 1] : 0.0f;
        const float old = ae[j];
        ae[j] = ANY ? bca_alpha_any(s_hi[j], s_nx[j], wgt(2 * q + 1), wgt(2 * q + 2), ao[j], a_next, M)
                    : bca_alpha(s_hi[j], s_nx[j], wgt(2 * q + 1), wgt(2 * q + 2), ao[j], a_next, M);
        chg = fmaxf(chg, fabsf(ae[j] - old));
      }
      xe[q] = ae[j];
    }
    __syncthreads();
    if (tol_mode && row_max(chg) <= P.tol) { met = true; break; }
  }
  if (!met && t == 0 && P.status) atomicOr(P.status, TK_FLAG_NOT_CONVERGED);
  // y_i = w_i - alpha_i + alpha_{i-1}; the even dual of pair q - 1 is read before the arrays become the stage
  float y_lo[H], y_hi[H];
#pragma unroll
  for (int j = 0; j < H; ++j) {
    const int q = t + j * T;
    const float a_im1 = q > 0 ? xe[q - 1] : 0.0f;
    y_lo[j] = ANY ? bca_output(M, s_lo[j], wgt(2 * q), a_im1, ao[j]) : wgt(2 * q) - ao[j] + a_im1;
    y_hi[j] = ANY ? bca_output(M, s_hi[j], wgt(2 * q + 1), ao[j], ae[j]) : wgt(2 * q + 1) - ae[j] + ao[j];
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < H; ++j) {
    const int q = t + j * T;
    if (2 * q < n) {
      const unsigned long long e = keys[pad(2 * q)];
      const int idx = un_idx(e);
      if (idx < n) stage[idx] = (ANY && M.mag && un_neg(e)) ? -y_lo[j] : y_lo[j];
    }
    if (2 * q + 1 < n) {
      const unsigned long long e = keys[pad(2 * q + 1)];
      const int idx = un_idx(e);
      if (idx < n) stage[idx] = (ANY && M.mag && un_neg(e)) ? -y_hi[j] : y_hi[j];
    }
  }
  __syncthreads();
  float* o_row = P.out + row * (long long)n;
  for (int i = t; i < n; i += T) { float q = stage[i]; if (P.mode == TK_TOPK) q *= __ldg(x_row + i); o_row[i] = q; }
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
}

// ------------------------------------------------------------------ rows of 16385..131072 elements
// keys, idx: the row-major result of the global-memory radix sort (keys as the complemented
// order-preserving words it sorts ascending, idx = original index of each rank).  Block c of a
// row's cluster owns ranks [c * kClusterSpan, (c + 1) * kClusterSpan).
constexpr int kClusterE = 16;
constexpr int kClusterT = 1024;
constexpr int kClusterSpan = kClusterE * kClusterT;

__global__ void __launch_bounds__(kClusterT, 1) tk_cluster_dykstra_kernel(const Problem P, const uint32_t* keys,
                                                                          const int32_t* idx) {
  namespace cg = cooperative_groups;
  constexpr int E = kClusterE, T = kClusterT;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ float xch_a[T], xch_b[T];
  const int t = threadIdx.x, n = P.n;
  const int C = (int)cluster.num_blocks(), c = (int)cluster.block_rank();
  const long long row = blockIdx.x / C;
  const Math M = make_math_q24(P);
  const int rank0 = (c * T + t) * E;
  const uint32_t* k_row = keys + row * (long long)n;
  float s[E], y[E];
#pragma unroll
  for (int i = 0; i < E; ++i) s[i] = (rank0 + i < n) ? key2f(~__ldg(k_row + rank0 + i)) : 0.0f;
  // The neighbour's slot is in this block's array, or in the adjacent block's through the cluster's
  // shared-memory window.  Every exchange is write, cluster barrier, read.  The solver alternates
  // the two kinds of exchange, and each has its own array: a thread overwrites its slot of one
  // array only after the barrier of the other kind's exchange, which every thread passes after
  // its read of the first.  So the solver's sync() between exchanges needs no barrier of its own
  // (two cluster barriers per sweep instead of four), except after the one exchange that precedes
  // the sweeps, which is followed by another of its kind.  A last barrier keeps every block
  // resident until its neighbours have read its arrays.
  const float* nxt_a = (c + 1 < C) ? cluster.map_shared_rank(xch_a, c + 1) : xch_a;
  const float* prv_b = (c > 0) ? cluster.map_shared_rank(xch_b, c - 1) : xch_b;
  const bool has_next = !(c == C - 1 && t == T - 1), has_prev = !(c == 0 && t == 0);
  auto next_of = [&](float x) -> float {
    xch_a[t] = x; cluster.sync();
    return (t + 1 < T) ? xch_a[t + 1] : (has_next ? nxt_a[0] : 0.0f);
  };
  auto prev_of = [&](float x) -> float {
    xch_b[t] = x; cluster.sync();
    return (t > 0) ? xch_b[t - 1] : (has_prev ? prv_b[T - 1] : 0.0f);
  };
  bool before_sweeps = true;
  auto sync = [&]() { if (before_sweeps) { cluster.sync(); before_sweeps = false; } };
  // 1024 threads leave 64 registers each: the keys are read again (L2) for the output map instead
  // of living through the sweeps, which keeps the iterate and its corrections out of local memory
  // (spill traffic was also what every cluster barrier's fence waited for)
  auto key_again = [&](int i) -> float { return (rank0 + i < n) ? key2f(~__ldg(k_row + rank0 + i)) : 0.0f; };
  // (a fixed number of sweeps only: the tolerance mode is served for rows of one thread block)
  solve_pairs<E, false>(P, M, s, rank0, has_next, has_prev, next_of, prev_of, sync, key_again,
                        [](float x) -> float { return x; }, y);
  cluster.sync();

  // un-permute: out[sigma_i] = y_i (times the sign of theta for the magnitude mode, times theta for
  // topk).  The row was just read by the sort, so these scattered accesses are served by L2.
  const int32_t* i_row = idx + row * (long long)n;
  const float* x_row = P.theta + row * (long long)n;
  float* o_row = P.out + row * (long long)n;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    if (rank0 + i >= n) continue;
    const int j = __ldg(i_row + rank0 + i);
    float q = y[i];
    if (M.mag || P.mode == TK_TOPK) {
      const float th = __ldg(x_row + j);
      if (M.mag) q = (__float_as_uint(th) >> 31) ? -q : q; else q *= th;
    }
    o_row[j] = q;
  }
}

}  // namespace

int cta_padded_length(int n);

int dykstra_cluster_max_n() { return 8 * kClusterSpan; }

// Alternating projections on rows already sorted into global memory (keys, idx as above).
cudaError_t launch_dykstra_cluster(const Problem& P, const uint32_t* keys, const int32_t* idx,
                                   cudaStream_t stream) {
  const int C = (P.n + kClusterSpan - 1) / kClusterSpan;
  if (C < 1 || C > 8) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(P.rows * C));
  cfg.blockDim = dim3(kClusterT);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tk_cluster_dykstra_kernel, P, keys, idx);
}

cudaError_t launch_dykstra(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  if (P.n <= 256) {
    int G = 1;
    while (G * EPL < P.n) G <<= 1;
    P.N = G * EPL;
    const long long groups = 128 / G;
    const unsigned blocks = (unsigned)((P.rows + groups - 1) / groups);
    const bool closed = P.q4 && P.mode != TK_TOPKMAG && !(P.qm1 > 0.0f);   // p = 4/3, phi = x: closed-form pair step
    const bool any = P.qm1 > 0.0f || (P.q4 && P.mode == TK_TOPKMAG);         // any other q != 2: root-solving pair step
    if (closed || any) {                       // dual coordinate ascent, pairs dealt round-robin to the row's lanes
#define TK_GROUP_BCA(GG)                                                     \
  do {                                                                       \
    if (any) tk_group_bca_kernel<GG, true><<<blocks, 128, 0, stream>>>(P);   \
    else tk_group_bca_kernel<GG, false><<<blocks, 128, 0, stream>>>(P);      \
  } while (0)
      switch (G) {
        case 1: TK_GROUP_BCA(1); break;
        case 2: TK_GROUP_BCA(2); break;
        case 4: TK_GROUP_BCA(4); break;
        case 8: TK_GROUP_BCA(8); break;
        case 16: TK_GROUP_BCA(16); break;
        default: TK_GROUP_BCA(32); break;
      }
#undef TK_GROUP_BCA
      return cudaGetLastError();
    }
    switch (G) {
      case 1: tk_group_dykstra_kernel<1><<<blocks, 128, 0, stream>>>(P); break;
      case 2: tk_group_dykstra_kernel<2><<<blocks, 128, 0, stream>>>(P); break;
      case 4: tk_group_dykstra_kernel<4><<<blocks, 128, 0, stream>>>(P); break;
      case 8: tk_group_dykstra_kernel<8><<<blocks, 128, 0, stream>>>(P); break;
      case 16: tk_group_dykstra_kernel<16><<<blocks, 128, 0, stream>>>(P); break;
      default: tk_group_dykstra_kernel<32><<<blocks, 128, 0, stream>>>(P); break;
    }
    return cudaGetLastError();
  }
  P.N = cta_padded_length(P.n);
  const int E = P.N >= 4096 ? 16 : (P.N >= 1024 ? 8 : 4);
  const int T = P.N / E;
  const size_t smem = (size_t)(P.N + (P.N >> PAD_SHIFT) + 1) * 8 + (size_t)(T + 2) * 8 + 16;
  void (*kern)(const Problem) = nullptr;
  int slot;
  switch (E) {
    case 4: kern = tk_cta_dykstra_kernel<4, 128>; slot = 0; break;
    case 8: kern = tk_cta_dykstra_kernel<8, 256>; slot = 1; break;
    default:
      if (T > 512) { kern = tk_cta_dykstra_kernel<16, 1024>; slot = 3; }
      else { kern = tk_cta_dykstra_kernel<16, 512>; slot = 2; }
      break;
  }
  size_t smem_used = smem;
  const bool closed = P.q4 && P.mode != TK_TOPKMAG && !(P.qm1 > 0.0f);
  const bool any = P.qm1 > 0.0f || (P.q4 && P.mode == TK_TOPKMAG);
  if (closed || any) {
    // q != 2: dual coordinate ascent with the pairs dealt round-robin (one dual per pair and family in shared memory)
    smem_used = (size_t)(P.N + (P.N >> PAD_SHIFT) + 1) * 8 + (size_t)P.N * 4 + 16;
    switch (E) {
      case 4: kern = any ? tk_cta_bca_kernel<4, 128, 4, true> : tk_cta_bca_kernel<4, 128, 6, false>; slot = 4; break;
      case 8: kern = any ? tk_cta_bca_kernel<8, 256, 2, true> : tk_cta_bca_kernel<8, 256, 3, false>; slot = 5; break;
      default:
        if (T > 512) { kern = any ? tk_cta_bca_kernel<16, 1024, 1, true> : tk_cta_bca_kernel<16, 1024, 1, false>; slot = 7; }
        else if (T > 256) { kern = any ? tk_cta_bca_kernel<16, 512, 1, true> : tk_cta_bca_kernel<16, 512, 1, false>; slot = 6; }
        else { kern = any ? tk_cta_bca_kernel<16, 256, 2, true> : tk_cta_bca_kernel<16, 256, 3, false>; slot = 8; }
        break;
    }
    if (any) slot += 5;
  }
  static bool configured[14][64] = {};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !configured[slot][dev]) {
    const int max_smem = (16384 + (16384 >> PAD_SHIFT) + 1) * 8 + 16384 * 4 + 16;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (err != cudaSuccess) return err;
    // several rows per SM need their shared memory at the same time
    cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (dev >= 0 && dev < 64) configured[slot][dev] = true;
  }
  kern<<<(unsigned)P.rows, (unsigned)T, smem_used, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace tk
