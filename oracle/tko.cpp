// tko.cpp -- CPU oracle for the p-norm-regularised top-k operators.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
// what the operators compute.  It exists so that the CUDA library can be
// checked against it; it is never part of the product path and shares no code
// with it.  Only the tests, the smoke check and the CPU-baseline leg of the
// benchmark may load it.
//
// What it computes, per row, following the paper in its own order:
//   1. key = theta (topkmask, topk) or |theta| (topkmag); sigma = stable
//      descending argsort of key, s = key_sigma        (Sec. 3, argsort/sort;
//      Prop. 5 and Prop. 6 "let sigma be the permutation sorting x / |x|").
//   2. w = (1,..,1,0,..,0) with k ones                  (Sec. 3, LP form of
//      the top-k mask, w = 1_k).
//   3. v* = argmin_{v_1>=..>=v_n} sum_i h_i(v_i),
//      h_i(v) = r*(s_i - v) + w_i phi(v)                (Sec. 5, separable
//      isotonic problem), by the pool-adjacent-violators procedure of
//      App. B.2: start from singletons at their own minimisers, merge two
//      adjacent blocks while the left value is strictly smaller than the
//      right one, re-solving the pooling sub-problem after each merge.
//   4. phi even: clip v at 0                            (Sec. 5, remark after
//      Prop. 6 on the non-negativity constraint).
//   5. y^s = (r*)'(s - v); un-permute (times sign(theta) for phi even); for
//      topk multiply the mask by theta                  (Prop. 2, Prop. 5/6).
//   6. VJP through the block structure                  (Prop. 7), chained
//      through step 5.
//   7. Alternating projections / dual block coordinate ascent on the odd and
//      even adjacent-pair constraints                   (Algorithm 1 and
//      App. A.8), fixed number of sweeps.
//
//   8. General sorted w (Sec. 3, LP forms of sort and rank over the
//      permutahedron P(w); Sec. 4, the relaxed operator for any w): tko_fwd_w /
//      tko_vjp_w run steps 1, 3, 5, 6 with phi(x) = x and the caller's
//      non-increasing w in place of 1_k; every pooled block is solved member by
//      member (closed form for p = 2).
//
// Regulariser: R(y) = (lambda/p) sum |y_i|^p (the form used in the paper's
// example after the PAV paragraph, in its Figure 3 and in its experiments),
// hence r*(t) = |t|^q / (q lambda^(q-1)), q = p/(p-1), and
// rho(t) := (r*)'(t) = sign(t) (|t|/lambda)^(q-1).
//
// Pooling sub-problem (App. A.6): p = 2 in closed form; q = 4 (p = 4/3) as the
// cubic the appendix states, its coefficients carried as power sums of the
// block members, then every pooled block of the final partition re-solved by
// summing over its members directly; any other p by summing over the members.
// TKO_FLAG_RESUM forces the member-by-member solve everywhere.
//
// parity unpinned: the relaxed *topk* (values of a signed input) has no
// definition in the paper beyond its hard limit; it is taken here as
// theta * topkmask_R(theta) and is pinned only through the mask oracle, the
// lambda -> 0 limit and finite differences.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <limits>
#include <numeric>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum Mode { MASK = 0, TOPK = 1, TOPKMAG = 2 };
enum Flags { FLAG_RESUM = 1, FLAG_SINGLE_THREAD = 2 };

struct Params {
  double p, q, lambda;
  bool mag;        // phi(x) = x^2/2 (true) or phi(x) = x (false)
  bool q_is_2, q_is_4;
};

Params make_params(double p, double lambda, int mode) {
  Params P;
  P.p = p;
  P.q = p / (p - 1.0);
  P.lambda = lambda;
  P.mag = (mode == TOPKMAG);
  P.q_is_2 = std::fabs(P.q - 2.0) < 1e-9;
  P.q_is_4 = std::fabs(P.q - 4.0) < 1e-9;
  if (P.q_is_2) P.q = 2.0;
  if (P.q_is_4) P.q = 4.0;
  return P;
}

// rho(t) = (r*)'(t) = sign(t) (|t|/lambda)^(q-1)
double rho(const Params& P, double t) {
  if (P.q_is_2) return t / P.lambda;
  double a = std::fabs(t) / P.lambda;
  double m = P.q_is_4 ? a * a * a : std::pow(a, P.q - 1.0);
  return t < 0 ? -m : m;
}

// rho'(t) = (q-1) |t|^(q-2) / lambda^(q-1)
double drho(const Params& P, double t) {
  if (P.q_is_2) return 1.0 / P.lambda;
  double a = std::fabs(t) / P.lambda;
  if (P.q_is_4) return 3.0 * a * a / P.lambda;
  if (a == 0.0) return P.q > 2.0 ? 0.0 : std::numeric_limits<double>::infinity();
  return (P.q - 1.0) * std::pow(a, P.q - 2.0) / P.lambda;
}

// inverse of rho on t >= 0: rho(t) = y  <=>  t = lambda y^(1/(q-1))
double rho_inv(const Params& P, double y) {
  if (P.q_is_2) return P.lambda * y;
  double a = std::fabs(y);
  double m = P.q_is_4 ? std::cbrt(a) : std::pow(a, 1.0 / (P.q - 1.0));
  return y < 0 ? -P.lambda * m : P.lambda * m;
}

// d/dgamma of sum_{i in [lo,hi)} h_i(gamma) = sum -rho(s_i - gamma) + w_i phi'(gamma)
double pooled_derivative(const Params& P, const double* s, int64_t lo, int64_t hi, int64_t k,
                         double gamma) {
  double acc = 0.0;
  for (int64_t i = lo; i < hi; ++i) {
    double w = i < k ? 1.0 : 0.0;
    acc += -rho(P, s[i] - gamma) + w * (P.mag ? gamma : 1.0);
  }
  return acc;
}

// Minimiser of the pooled objective over members [lo,hi) (0-based sorted
// ranks), found by bisection on its increasing derivative.
// Bracket: the derivative is >= 0 at max s, and <= 0 at min s - lambda
// (phi = x: rho(s_i - gamma) >= rho(lambda) = 1 >= w_i) or at 0 (phi even,
// s >= 0: every term is <= 0).
double solve_block_by_members(const Params& P, const double* s, int64_t lo, int64_t hi,
                              int64_t k) {
  double smax = s[lo], smin = s[hi - 1];
  double a = P.mag ? std::min(0.0, smin) : smin - P.lambda;
  double b = smax;
  if (pooled_derivative(P, s, lo, hi, k, b) <= 0.0) return b;
  if (pooled_derivative(P, s, lo, hi, k, a) >= 0.0) return a;
  for (int it = 0; it < 400; ++it) {
    double m = 0.5 * (a + b);
    if (m <= a || m >= b) break;
    if (pooled_derivative(P, s, lo, hi, k, m) > 0.0) b = m; else a = m;
  }
  return 0.5 * (a + b);
}

struct Block {
  int64_t lo, hi;          // members: sorted ranks [lo, hi)
  double gamma;
  long double S1, S2, S3;  // power sums of the members' s (closed-form solves)
};

// Root of the monotone cubic of App. A.6 from the block's power sums:
//   sum (gamma - s_i)^3 + lambda^3 m_B          = 0   (phi = x)
//   sum (gamma - s_i)^3 + lambda^3 m_B gamma    = 0   (phi even)
// with sum (gamma - s_i)^3 = N gamma^3 - 3 S1 gamma^2 + 3 S2 gamma - S3.
double solve_cubic_from_sums(const Params& P, const Block& B, int64_t k, double smin, double smax) {
  long double N = (long double)(B.hi - B.lo);
  long double m = (long double)std::max<int64_t>(0, std::min(B.hi, k) - B.lo);
  long double l3 = (long double)P.lambda * P.lambda * P.lambda;
  auto f = [&](long double g) -> long double {
    long double poly = ((N * g - 3.0L * B.S1) * g + 3.0L * B.S2) * g - B.S3;
    return poly + (P.mag ? l3 * m * g : l3 * m);
  };
  long double a = P.mag ? std::min(0.0, smin) : smin - P.lambda;
  long double b = smax;
  if (f(b) <= 0) return (double)b;
  if (f(a) >= 0) return (double)a;
  for (int it = 0; it < 400; ++it) {
    long double mid = 0.5L * (a + b);
    if (mid <= a || mid >= b) break;
    if (f(mid) > 0) b = mid; else a = mid;
  }
  return (double)(0.5L * (a + b));
}

double solve_block(const Params& P, const double* s, const Block& B, int64_t k, bool resum) {
  int64_t N = B.hi - B.lo;
  int64_t m = std::max<int64_t>(0, std::min(B.hi, k) - B.lo);
  if (!resum && P.q_is_2) {
    // App. A.6 / the example of Sec. 5: gamma = sum s / sum (lambda w + 1) for
    // phi even; for phi = x the derivative sum (gamma - s_i)/lambda + w_i
    // vanishes at gamma = (sum s - lambda m) / N.
    if (P.mag) return (double)(B.S1 / ((long double)N + (long double)P.lambda * m));
    return (double)((B.S1 - (long double)P.lambda * m) / (long double)N);
  }
  if (!resum && P.q_is_4 && N > 1) return solve_cubic_from_sums(P, B, k, s[B.hi - 1], s[B.lo]);
  if (N == 1 && !P.mag) {
    // singleton, phi = x: rho(s - v) = w  =>  v = s - lambda w^(1/(q-1)), w in {0,1}
    return B.lo < k ? s[B.lo] - P.lambda : s[B.lo];
  }
  if (N == 1 && P.mag && B.lo >= k) return s[B.lo];   // w = 0: h = r*(s - v), minimised at v = s
  return solve_block_by_members(P, s, B.lo, B.hi, k);
}

// Pool adjacent violators (App. B.2).  Blocks are kept on a stack in rank
// order; a new singleton is pushed with its own minimiser and the two top
// blocks are merged while the earlier one has a strictly smaller value.
void pav(const Params& P, const double* s, int64_t n, int64_t k, bool resum,
         std::vector<Block>& blocks) {
  blocks.clear();
  blocks.reserve(n);
  for (int64_t i = 0; i < n; ++i) {
    Block b;
    b.lo = i; b.hi = i + 1;
    b.S1 = s[i]; b.S2 = (long double)s[i] * s[i]; b.S3 = b.S2 * s[i];
    b.gamma = solve_block(P, s, b, k, resum);
    blocks.push_back(b);
    while (blocks.size() >= 2) {
      Block& prev = blocks[blocks.size() - 2];
      Block& last = blocks[blocks.size() - 1];
      if (!(prev.gamma < last.gamma)) break;
      prev.hi = last.hi;
      prev.S1 += last.S1; prev.S2 += last.S2; prev.S3 += last.S3;
      blocks.pop_back();
      Block& merged = blocks.back();
      merged.gamma = solve_block(P, s, merged, k, resum);
    }
  }
  if (!resum && P.q_is_4) {
    // the partition is settled; re-solve every pooled block over its members
    for (Block& b : blocks)
      if (b.hi - b.lo > 1) b.gamma = solve_block_by_members(P, s, b.lo, b.hi, k);
  }
}

// stable descending argsort of the key, ties in ascending index
void argsort_row(const float* theta, int64_t n, bool mag, int32_t* perm, double* s) {
  std::vector<double> key(n);
  for (int64_t i = 0; i < n; ++i) key[i] = mag ? std::fabs((double)theta[i]) : (double)theta[i];
  std::iota(perm, perm + n, 0);
  std::stable_sort(perm, perm + n, [&](int32_t a, int32_t b) { return key[a] > key[b]; });
  for (int64_t i = 0; i < n; ++i) s[i] = key[perm[i]];
}

struct RowWork {
  std::vector<int32_t> perm;
  std::vector<double> s, v, ys;
  std::vector<Block> blocks;
};

void forward_sorted(const Params& P, const float* theta, int64_t n, int64_t k, bool resum,
                    RowWork& W) {
  W.perm.resize(n); W.s.resize(n); W.v.resize(n); W.ys.resize(n);
  argsort_row(theta, n, P.mag, W.perm.data(), W.s.data());
  pav(P, W.s.data(), n, k, resum, W.blocks);
  for (const Block& b : W.blocks)
    for (int64_t i = b.lo; i < b.hi; ++i) W.v[i] = b.gamma;
  if (P.mag)
    for (int64_t i = 0; i < n; ++i) W.v[i] = std::max(W.v[i], 0.0);
  for (int64_t i = 0; i < n; ++i) W.ys[i] = rho(P, W.s[i] - W.v[i]);
}

inline double sign_of(float x) { return std::signbit(x) && x != 0.0f ? -1.0 : 1.0; }

int check_args(int64_t rows, int64_t n, int64_t k, double p, double lambda, int mode) {
  if (rows < 0 || n < 1 || k < 1 || k > n) return 1;
  if (!(p > 1.0) || !(lambda > 0.0)) return 1;
  if (mode < 0 || mode > 2) return 1;
  return 0;
}

}  // namespace

extern "C" {

int tko_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// perm[r*n + i] = original index of the i-th largest key of row r; sorted (may
// be NULL) receives the keys in that order.
int tko_argsort(const float* theta, int64_t rows, int64_t n, int mode, int32_t* perm,
                double* sorted) {
  if (rows < 0 || n < 1 || mode < 0 || mode > 2) return 1;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<double> s(n);
    argsort_row(theta + r * n, n, mode == TOPKMAG, perm + r * n, s.data());
    if (sorted) std::copy(s.begin(), s.end(), sorted + r * n);
  }
  return 0;
}

// Forward pass.  out: [rows*n] operator output.  Optional (NULL to skip):
// perm [rows*n] sorting permutation; v [rows*n] isotonic solution in sorted
// coordinates; block_lo / block_hi [rows*n]: for every sorted rank the bounds
// [lo,hi) of the PAV block it ended in.
int tko_fwd(const float* theta, int64_t rows, int64_t n, int64_t k, double p, double lambda,
            int mode, int flags, double* out, int32_t* perm, double* v, int32_t* block_lo,
            int32_t* block_hi) {
  if (check_args(rows, n, k, p, lambda, mode)) return 1;
  const Params P = make_params(p, lambda, mode);
  const bool resum = (flags & FLAG_RESUM) != 0;
  const bool single = (flags & FLAG_SINGLE_THREAD) != 0;
#pragma omp parallel if (!single)
  {
    RowWork W;
#pragma omp for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
      const float* x = theta + r * n;
      forward_sorted(P, x, n, k, resum, W);
      double* y = out + r * n;
      for (int64_t i = 0; i < n; ++i) {
        int32_t j = W.perm[i];
        double val = W.ys[i];
        if (mode == TOPKMAG) val *= sign_of(x[j]);
        if (mode == TOPK) val *= (double)x[j];
        y[j] = val;
      }
      if (perm) std::copy(W.perm.begin(), W.perm.end(), perm + r * n);
      if (v) std::copy(W.v.begin(), W.v.end(), v + r * n);
      if (block_lo && block_hi)
        for (const Block& b : W.blocks)
          for (int64_t i = b.lo; i < b.hi; ++i) {
            block_lo[r * n + i] = (int32_t)b.lo;
            block_hi[r * n + i] = (int32_t)b.hi;
          }
    }
  }
  return 0;
}

// Vector-Jacobian product grad = J^T g of the forward map at theta.
// In sorted coordinates, with t_j = s_j - v_j and rho'_j = rho'(t_j), Prop. 7
// gives for a block B: d gamma_B / d s_j = rho'_j / D_B,
// D_B = sum_B rho'_l (+ m_B for phi even, m_B = number of members with w = 1;
// with lambda inside R the w_j of the printed formula is multiplied by
// lambda^(q-1), which is what rho' carrying the lambda expresses).
// Chaining through y^s_i = rho(s_i - gamma_B):
//   o_j = rho'_j (g^s_j - A_B / D_B),  A_B = sum_B rho'_l g^s_l,
// and o_j = 0 where D_B = 0 (the 0/0 case of a w = 0 singleton with q > 2).
int tko_vjp(const float* theta, const float* gout, int64_t rows, int64_t n, int64_t k, double p,
            double lambda, int mode, int flags, double* grad) {
  if (check_args(rows, n, k, p, lambda, mode)) return 1;
  const Params P = make_params(p, lambda, mode);
  const bool resum = (flags & FLAG_RESUM) != 0;
  const bool single = (flags & FLAG_SINGLE_THREAD) != 0;
#pragma omp parallel if (!single)
  {
    RowWork W;
    std::vector<double> gs, o;
#pragma omp for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
      const float* x = theta + r * n;
      const float* g = gout + r * n;
      forward_sorted(P, x, n, k, resum, W);
      gs.assign(n, 0.0); o.assign(n, 0.0);
      for (int64_t i = 0; i < n; ++i) {
        int32_t j = W.perm[i];
        double chi = 1.0;
        if (mode == TOPKMAG) chi = sign_of(x[j]);
        if (mode == TOPK) chi = (double)x[j];
        gs[i] = chi * (double)g[j];
      }
      for (const Block& b : W.blocks) {
        double D = 0.0, A = 0.0;
        int64_t m = std::max<int64_t>(0, std::min(b.hi, k) - b.lo);
        for (int64_t i = b.lo; i < b.hi; ++i) {
          double d = drho(P, W.s[i] - W.v[i]);
          D += d; A += d * gs[i];
        }
        if (P.mag) D += (double)m;
        for (int64_t i = b.lo; i < b.hi; ++i) {
          double d = drho(P, W.s[i] - W.v[i]);
          o[i] = (D > 0.0) ? d * (gs[i] - A / D) : 0.0;
        }
      }
      double* gr = grad + r * n;
      for (int64_t i = 0; i < n; ++i) {
        int32_t j = W.perm[i];
        double val = o[i];
        if (mode == TOPKMAG) val *= sign_of(x[j]);
        if (mode == TOPK) val += (double)g[j] * W.ys[i];   // product rule: g * mask
        gr[j] = val;
      }
    }
  }
  return 0;
}

// Alternating projections on C1 (pairs (1,2),(3,4),..) and C2 (pairs (2,3),
// (4,5),..), `sweeps` full iterations, no early exit.
//
// p = 2 (Algorithm 1).  The objective sum h_i is, up to a constant,
// 1/2 sum c_i (v_i - z_i)^2 / lambda with c_i = 1, z_i = s_i - lambda w_i for
// phi = x and c_i = 1 + lambda w_i, z_i = s_i / c_i for phi even, so v* is the
// projection of z onto C1 n C2 in the metric c.  Dykstra's iteration is run on
// z with plain projections: y = Proj_C1(v + p), p <- v + p - y,
// v = Proj_C2(y + q), q <- y + q - v; a pair (a, b) that violates a >= b is
// replaced by its c-weighted mean.  (Read literally, Algorithm 1 starts at s
// and subtracts w inside *both* half-steps; that iteration converges to the
// projection of s - 2w -- for n = 1 it returns s - 2w after one iteration --
// so the linear term is applied once, by starting from z.)
//
// p != 2 (App. A.8): block coordinate ascent on the duals alpha_1..alpha_{n-1}
// (alpha_0 = alpha_n = 0), odd coordinates then even coordinates.  Each
// coordinate solves its two-variable primal sub-problem
//   min_{v_i >= v_{i+1}} h_i(v_i) + h_{i+1}(v_{i+1}) + alpha_{i-1} v_i - alpha_{i+1} v_{i+1};
// unconstrained minimisers are kept when ordered (alpha_i = 0), otherwise both
// are set to the common minimiser gamma and alpha_i = h_i'(gamma) + alpha_{i-1}
// with the sign convention h_i'(v_i) + alpha_{i-1} - alpha_i = 0.  The primal
// iterate is v_i = argmin_v h_i(v) + (alpha_{i-1} - alpha_i) v.
static double shifted_minimiser(const Params& P, double s, double w, double c) {
  // argmin_v r*(s - v) + w phi(v) + c v :  -rho(s - v) + w phi'(v) + c = 0
  if (!P.mag) return s - rho_inv(P, w + c);
  // phi even: -rho(s - v) + w v + c increasing in v; bisection
  auto f = [&](double v) { return -rho(P, s - v) + w * v + c; };
  double span = std::fabs(s) + P.lambda * (1.0 + std::fabs(c)) + std::fabs(c) + 1.0;
  double a = s - span, b = s + span;
  for (int grow = 0; grow < 200 && f(a) > 0; ++grow) { span *= 2; a = s - span; }
  for (int grow = 0; grow < 200 && f(b) < 0; ++grow) { span *= 2; b = s + span; }
  for (int it = 0; it < 400; ++it) {
    double m = 0.5 * (a + b);
    if (m <= a || m >= b) break;
    if (f(m) > 0) b = m; else a = m;
  }
  return 0.5 * (a + b);
}

static double pair_common_minimiser(const Params& P, double s1, double w1, double c1, double s2,
                                    double w2, double c2, double lo, double hi) {
  auto f = [&](double g) {
    return -rho(P, s1 - g) + w1 * (P.mag ? g : 1.0) + c1 - rho(P, s2 - g) +
           w2 * (P.mag ? g : 1.0) + c2;
  };
  double a = lo, b = hi;   // the common minimiser lies between the two separate minimisers
  for (int it = 0; it < 400; ++it) {
    double m = 0.5 * (a + b);
    if (m <= a || m >= b) break;
    if (f(m) > 0) b = m; else a = m;
  }
  return 0.5 * (a + b);
}

int tko_dykstra(const float* theta, int64_t rows, int64_t n, int64_t k, double p, double lambda,
                int mode, int sweeps, int flags, double* out, double* v_out) {
  if (check_args(rows, n, k, p, lambda, mode) || sweeps < 0) return 1;
  const Params P = make_params(p, lambda, mode);
  const bool single = (flags & FLAG_SINGLE_THREAD) != 0;
#pragma omp parallel if (!single)
  {
    std::vector<int32_t> perm(n);
    std::vector<double> s(n), v(n), y(n), pc(n), qc(n), c(n), alpha(n + 1);
#pragma omp for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
      const float* x = theta + r * n;
      argsort_row(x, n, P.mag, perm.data(), s.data());
      auto w = [&](int64_t i) { return i < k ? 1.0 : 0.0; };
      if (P.q_is_2) {
        for (int64_t i = 0; i < n; ++i) {
          c[i] = P.mag ? 1.0 + lambda * w(i) : 1.0;
          v[i] = P.mag ? s[i] / c[i] : s[i] - lambda * w(i);
          pc[i] = qc[i] = 0.0;
        }
        auto project = [&](const std::vector<double>& in, std::vector<double>& res, int64_t first) {
          res = in;
          for (int64_t i = first; i + 1 < n; i += 2)
            if (in[i] < in[i + 1]) {
              double mean = (c[i] * in[i] + c[i + 1] * in[i + 1]) / (c[i] + c[i + 1]);
              res[i] = res[i + 1] = mean;
            }
        };
        std::vector<double> tmp(n);
        for (int it = 0; it < sweeps; ++it) {
          for (int64_t i = 0; i < n; ++i) tmp[i] = v[i] + pc[i];
          project(tmp, y, 0);
          for (int64_t i = 0; i < n; ++i) pc[i] = tmp[i] - y[i];
          for (int64_t i = 0; i < n; ++i) tmp[i] = y[i] + qc[i];
          project(tmp, v, 1);
          for (int64_t i = 0; i < n; ++i) qc[i] = tmp[i] - v[i];
        }
      } else {
        // alpha[i] for i = 1..n-1 is the multiplier of v_i >= v_{i+1} (1-based)
        std::fill(alpha.begin(), alpha.end(), 0.0);
        auto update = [&](int64_t i) {   // 1-based constraint index, 1 <= i <= n-1
          double s1 = s[i - 1], s2 = s[i], w1 = w(i - 1), w2 = w(i);
          double c1 = alpha[i - 1], c2 = -alpha[i + 1];
          double v1 = shifted_minimiser(P, s1, w1, c1);
          double v2 = shifted_minimiser(P, s2, w2, c2);
          if (v1 >= v2) { alpha[i] = 0.0; return; }
          double g = pair_common_minimiser(P, s1, w1, c1, s2, w2, c2, v1, v2);
          double hprime = -rho(P, s1 - g) + w1 * (P.mag ? g : 1.0);
          alpha[i] = std::max(0.0, hprime + alpha[i - 1]);
        };
        for (int it = 0; it < sweeps; ++it) {
          for (int64_t i = 1; i <= n - 1; i += 2) update(i);
          for (int64_t i = 2; i <= n - 1; i += 2) update(i);
        }
        for (int64_t i = 1; i <= n; ++i)
          v[i - 1] = shifted_minimiser(P, s[i - 1], w(i - 1), alpha[i - 1] - alpha[i]);
      }
      double* yo = out + r * n;
      for (int64_t i = 0; i < n; ++i) {
        double vi = P.mag ? std::max(v[i], 0.0) : v[i];
        int32_t j = perm[i];
        double val = rho(P, s[i] - vi);
        if (mode == TOPKMAG) val *= sign_of(x[j]);
        if (mode == TOPK) val *= (double)x[j];
        yo[j] = val;
        if (v_out) v_out[r * n + i] = vi;
      }
    }
  }
  return 0;
}

}  // extern "C"

// ---------------------------------------------------------------- general sorted w
// Relaxed linear maximisation over the permutahedron P(w) (Sec. 4 with phi(x) = x):
//   y_R(x, w) = argmax_{y in P(w)} <x, y> - R(y) = grad R*(x - u*),   u* = v*_{sigma^-1},
//   v* = argmin_{v_1 >= .. >= v_n} sum_i r*(s_i - v_i) + w_i v_i       (Prop. 5),
// w_1 >= .. >= w_n any real numbers.  With w = 1_k this is the relaxed top-k mask; with
// w = rho = (n, .., 1) and x -> -x the relaxed rank; with x = rho and w = sort(x) the relaxed sort
// (Sec. 3, LP forms).
namespace {

struct WBlock {
  int64_t lo, hi;
  double gamma;
};

// d/dgamma of sum_{i in [lo,hi)} r*(s_i - gamma) + w_i gamma = sum -rho(s_i - gamma) + w_i
double pooled_derivative_w(const Params& P, const double* s, const double* w, int64_t lo, int64_t hi,
                           double gamma) {
  double acc = 0.0;
  for (int64_t i = lo; i < hi; ++i) acc += -rho(P, s[i] - gamma) + w[i];
  return acc;
}

// Minimiser of the pooled objective: the derivative is increasing in gamma; each term vanishes at
// s_i - rho^-1(w_i), so the root lies between the smallest and the largest of those.
double solve_block_w(const Params& P, const double* s, const double* w, int64_t lo, int64_t hi) {
  if (P.q_is_2) {
    double ss = 0.0, ww = 0.0;
    for (int64_t i = lo; i < hi; ++i) { ss += s[i]; ww += w[i]; }
    return (ss - P.lambda * ww) / (double)(hi - lo);
  }
  double a = std::numeric_limits<double>::infinity(), b = -a;
  for (int64_t i = lo; i < hi; ++i) {
    double z = s[i] - rho_inv(P, w[i]);
    a = std::min(a, z); b = std::max(b, z);
  }
  if (hi - lo == 1) return a;
  for (int it = 0; it < 400; ++it) {
    double m = 0.5 * (a + b);
    if (m <= a || m >= b) break;
    if (pooled_derivative_w(P, s, w, lo, hi, m) > 0.0) b = m; else a = m;
  }
  return 0.5 * (a + b);
}

// Pool adjacent violators (App. B.2) for general w: the same stack of blocks, merge while the
// earlier of the two top blocks has a strictly smaller value, re-solve after each merge.
void pav_w(const Params& P, const double* s, const double* w, int64_t n, std::vector<WBlock>& blocks) {
  blocks.clear();
  for (int64_t i = 0; i < n; ++i) {
    WBlock b{i, i + 1, solve_block_w(P, s, w, i, i + 1)};
    blocks.push_back(b);
    while (blocks.size() >= 2) {
      WBlock& prev = blocks[blocks.size() - 2];
      WBlock& last = blocks[blocks.size() - 1];
      if (!(prev.gamma < last.gamma)) break;
      prev.hi = last.hi;
      blocks.pop_back();
      WBlock& merged = blocks.back();
      merged.gamma = solve_block_w(P, s, w, merged.lo, merged.hi);
    }
  }
}

int check_args_w(int64_t rows, int64_t n, double p, double lambda, const double* w, int64_t w_rows) {
  if (rows < 0 || n < 1 || !(p > 1.0) || !(lambda > 0.0) || w == nullptr) return 1;
  if (w_rows != 1 && w_rows != rows) return 1;
  for (int64_t r = 0; r < w_rows; ++r)
    for (int64_t i = 0; i + 1 < n; ++i)
      if (!(w[r * n + i] >= w[r * n + i + 1])) return 1;     // must be sorted (Prop. 1: "if not, sort w")
  return 0;
}

}  // namespace

extern "C" {

// out[r, :] = y_R(theta[r, :], w[r or 0, :]).  w: [w_rows * n] doubles, w_rows = 1 (shared) or rows,
// every row non-increasing.  Optional outputs as in tko_fwd.
int tko_fwd_w(const float* theta, const double* w, int64_t rows, int64_t n, int64_t w_rows, double p,
              double lambda, double* out, int32_t* perm, double* v, int32_t* block_lo, int32_t* block_hi) {
  if (check_args_w(rows, n, p, lambda, w, w_rows)) return 1;
  const Params P = make_params(p, lambda, MASK);
#pragma omp parallel
  {
    std::vector<int32_t> pm(n);
    std::vector<double> s(n);
    std::vector<WBlock> blocks;
#pragma omp for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
      const float* x = theta + r * n;
      const double* wr = w + (w_rows == 1 ? 0 : r) * n;
      argsort_row(x, n, false, pm.data(), s.data());
      pav_w(P, s.data(), wr, n, blocks);
      for (const WBlock& b : blocks)
        for (int64_t i = b.lo; i < b.hi; ++i) {
          out[r * n + pm[i]] = rho(P, s[i] - b.gamma);
          if (v) v[r * n + i] = b.gamma;
          if (block_lo) block_lo[r * n + i] = (int32_t)b.lo;
          if (block_hi) block_hi[r * n + i] = (int32_t)b.hi;
        }
      if (perm) std::copy(pm.begin(), pm.end(), perm + r * n);
    }
  }
  return 0;
}

// grad_theta = J^T g of y_R(., w) at theta (Prop. 7 with phi(x) = x: D_B = sum_B rho', no w term),
// chained through y^s_i = rho(s_i - gamma_B): o_j = rho'_j (g^s_j - A_B / D_B), 0 where D_B = 0.
// grad_w (may be null): the cotangent pulled back to w, per row and in w's own (sorted) order.  Inside a
// pooled block B the value gamma solves sum_B rho(s_i - gamma) = sum_B w_i (stationarity of the block, Prop. 5
// with phi(x) = x), so d gamma / d w_j = -1 / D_B and d y_i / d w_j = rho'_i / D_B for i, j in B: the pulled-back
// cotangent of every w_j of the block is A_B / D_B.  A singleton has y_j = w_j: its entry is g_j also where
// rho' vanishes.
int tko_vjp_w(const float* theta, const double* w, const float* gout, int64_t rows, int64_t n,
              int64_t w_rows, double p, double lambda, double* grad, double* grad_w) {
  if (check_args_w(rows, n, p, lambda, w, w_rows)) return 1;
  const Params P = make_params(p, lambda, MASK);
#pragma omp parallel
  {
    std::vector<int32_t> pm(n);
    std::vector<double> s(n);
    std::vector<WBlock> blocks;
#pragma omp for schedule(dynamic, 4)
    for (int64_t r = 0; r < rows; ++r) {
      const float* x = theta + r * n;
      const float* g = gout + r * n;
      const double* wr = w + (w_rows == 1 ? 0 : r) * n;
      argsort_row(x, n, false, pm.data(), s.data());
      pav_w(P, s.data(), wr, n, blocks);
      for (const WBlock& b : blocks) {
        double D = 0.0, A = 0.0;
        for (int64_t i = b.lo; i < b.hi; ++i) {
          double d = drho(P, s[i] - b.gamma);
          D += d; A += d * (double)g[pm[i]];
        }
        for (int64_t i = b.lo; i < b.hi; ++i) {
          double d = drho(P, s[i] - b.gamma);
          grad[r * n + pm[i]] = (D > 0.0) ? d * ((double)g[pm[i]] - A / D) : 0.0;
          if (grad_w)
            grad_w[r * n + i] = (D > 0.0) ? A / D : (b.hi - b.lo == 1 ? (double)g[pm[i]] : 0.0);
        }
      }
    }
  }
  return 0;
}

}  // extern "C"
