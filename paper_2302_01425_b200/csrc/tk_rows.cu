// tk_rows.cu -- rows of up to 1024 elements, the default forward pass and VJP.
//
// Every warp works alone on its rows (up to 32 of them for n <= 64, one warp per row with 1 to 8
// rows per warp for n > 128), in three phases:
//   1. in batches of 32/G rows (G lanes per row with 8 keys each up to n = 256, a warp per row with
//      16 or 32 keys per lane above; one lane with 16 keys for 8 < n <= 16, where the whole
//      network runs in registers): load, sort the 32-bit KEYS by the shuffle network, leave the
//      sorted row in the warp's shared memory;
//   2. the isotonic problem of Sec. 5 has at most one pooled block [a0, b0) around ranks k-1 and
//      k, and it is grown from that pair, pooling a neighbour while it violates the order, on
//      running power sums of d = key - pivot.  Lane r grows row r one rank at a time
//      (solve_row_walk): up to 32 rows side by side, a few instructions per block member, instead
//      of a search replicated over the lanes of every row.  A warp that owns whole rows whose
//      window is wide grows them together, 32 candidates per step (solve_row_coop);
//   3. in the same batches: the results by value (given gamma and the cap width, the output and
//      the VJP of an element depend on its own key alone), stored where they were loaded.
// No index travels through the sort and nothing is scattered; the phases are separated by warp
// barriers only, so the other warps of the SM fill the latency of a warp that is growing a block.
// The block value is solved in fp32 about the block mean (App. A.6 cubic in depressed form).
#include "tk_common.cuh"
#include "tk_group_sort.cuh"
#include "tk_key_sort.cuh"

namespace tk {

namespace {

struct RowSol { float piv, u, c; int a0, b0, has_block; };

// Root u of the pooled block's stationarity equation, about the block mean mu (d = key - pivot,
// M2, M3 the central sums of the cnt members, m of them with w = 1):
//   q = 2, phi = x  : sum (d_i - u) = lam m                 q = 2, phi even: ... = lam m (piv + u)
//   q = 4, phi = x  : sum (d_i - u)^3 = lam^3 m             q = 4, phi even: ... = lam^3 m (piv + u)
// With w = u - mu the cubic is w^3 + P w + Q = 0, P >= 0: one real root, by Cardano in the form
// without cancellation (the two cube roots multiply to -P/3), polished by two Newton steps.
template <bool Q4, bool MAG>
__device__ __forceinline__ float block_value(float lam, float lam3, float piv, float cnt, float m,
                                             float mu, float M2, float M3) {
  if (!Q4) return MAG ? (cnt * mu - lam * m * piv) / (cnt + lam * m) : mu - lam * m / cnt;
  const float l3m = lam3 * m;
  const float inv = 1.0f / cnt;
  const float Pc = (3.0f * M2 + (MAG ? l3m : 0.0f)) * inv;
  const float Qc = (l3m * (MAG ? piv + mu : 1.0f) - M3) * inv;
  const float third = Pc * (1.0f / 3.0f);
  const float Rt = sqrtf(0.25f * Qc * Qc + third * third * third);
  const float A = cbrtf(0.5f * fabsf(Qc) + Rt);
  const float B = (A != 0.0f) ? third / A : 0.0f;
  const float den = A * A + third + B * B;
  float w = (den > 0.0f) ? -Qc / den : 0.0f;
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const float fp = fmaf(3.0f * w, w, Pc);
    if (fp > 0.0f) w -= fmaf(fmaf(w, w, Pc), w, Qc) / fp;
  }
  return mu + w;
}

// The isotonic solve of one row by ONE thread, on the row's sorted keys in shared memory (rank i at
// sk[i]).  With w = 1_k every rank is its own minimiser (vtop(s_i) for i < k, s_i for i >= k) and
// both runs are non-increasing, so pooling adjacent violators only ever grows ONE block from the
// pair (k-1, k) (Sec. 5).  The block [a, b) with m = k - a weighted members has the value gamma
// that solves  H(tau) = sum_{i in block} rho(s_i - tau) - m phi'(tau) = 0,  H decreasing, and
//   rank b   violates (gamma < s_b)          <=>  H(s_b) < 0          -> pool it,
//   rank a-1 violates (vtop(s_{a-1}) < gamma) <=>  H(vtop(s_{a-1})) > 0 -> pool it.
// rho is an odd polynomial of degree q - 1, so H is a polynomial in tau whose coefficients are the
// block's power sums of d = key - pivot: a test is a handful of fmas and pooling a rank is one add
// per sum.  The loop is flat (one candidate per step, the side changes when a test fails, two
// failures in a row end it), so 32 lanes with different rows stay in one instruction stream, and
// it runs for (block size + a few) steps.  The sums only ever grow; fp64 copies of them give the
// block mean and central moments for the block value.
template <bool Q4, bool MAG>
__device__ __forceinline__ void solve_row_walk(const float* sk, int n, int k, const Math& M, const Problem& P,
                                               RowSol& R) {
  auto key = [&](int i) -> float { return sk[i]; };
  const float c = key(k - 1);
  const float vtop_c = M.vtop(c);
  const bool has_block = (k < n) && (vtop_c < key(k));
  // Pivot for the arithmetic around the pooled block: its keys lie in (vtop(c), c + width(c)), so
  // differences from c are exact while that window stays within a factor two of c; for phi even
  // and large lambda the window reaches far below c and the keys themselves are well scaled.
  const float piv = (MAG && vtop_c < 0.5f * c) ? 0.0f : c;
  int a0 = k, b0 = k;
  float u = 0.0f;
  if (has_block) {
    const float il3 = P.inv_lam * P.inv_lam * P.inv_lam;
    float D1 = 0.f, D2 = 0.f, D3 = 0.f;
    double E1 = 0.0, E2 = 0.0, E3 = 0.0;
    auto pool = [&](float d) {
      D1 += d;
      const double dd = (double)d;
      E1 += dd;
      if (Q4) {
        const float d2 = d * d;
        D2 += d2; D3 = fmaf(d2, d, D3);
        const double dd2 = dd * dd;
        E2 += dd2; E3 = fma(dd2, dd, E3);
      }
    };
    // H at tau = pivot + uu for the block [a, b)
    auto H = [&](float uu, int a, int b) -> float {
      const float cnt = (float)(b - a), m = (float)(k - a);
      float S;
      if (Q4) S = (((-cnt * uu + 3.0f * D1) * uu - 3.0f * D2) * uu + D3) * il3;
      else S = (D1 - cnt * uu) * P.inv_lam;
      return S - (MAG ? m * (piv + uu) : m);
    };
    a0 = k - 1; b0 = k + 1;
    pool(c - piv);
    pool(key(k) - piv);
    int below = 1, fails = 0;          // which neighbour is tried next: rank b0 (below) or rank a0 - 1
    while (fails < 2) {
      bool joins = false;
      float d = 0.0f;
      if (below) {
        if (b0 < n) { d = key(b0) - piv; joins = H(d, a0, b0) < 0.0f; }
        b0 += joins ? 1 : 0;
      } else {
        if (a0 > 0) { const float s = key(a0 - 1); d = s - piv; joins = H(M.vtop(s) - piv, a0, b0) > 0.0f; }
        a0 -= joins ? 1 : 0;
      }
      if (joins) { pool(d); fails = 0; }
      else { ++fails; below ^= 1; }
    }
    // ---- block value from the mean and the central moments
    const double cntd = (double)(b0 - a0);
    const double mud = E1 / cntd;
    float M2 = 0.f, M3 = 0.f;
    if (Q4) {
      M2 = (float)(E2 - E1 * mud);
      M3 = (float)(E3 - 3.0 * mud * E2 + 2.0 * mud * mud * E1);
    }
    u = block_value<Q4, MAG>(P.lam, P.lam3, piv, (float)cntd, (float)(k - a0), (float)mud, M2, M3);
    u = settle_offset(M, piv, u, a0, b0, n, key);
  }
  R.piv = piv; R.u = u; R.c = c; R.a0 = a0; R.b0 = b0; R.has_block = has_block ? 1 : 0;
}

// Any other q (rho(t) = (t/lambda)^(q-1) through powf; mask and top-k modes): H is no polynomial, so
// the block is not grown but gamma is found as the root of the threshold function
//   F(tau) = #{s_i >= tau + lambda} - k + sum_{tau < s_i < tau + lambda} rho(s_i - tau)
// by one thread on its sorted row: safeguarded Newton inside the bracket (s_{k-1} - lambda, s_k),
// every pass over the window ranks only (those between the bracket's ends and a cap above), one
// Newton step on the current set's equation sum rho = m per pass, bisection when the step leaves
// the bracket.  The pass that sees the set it was computed from and has a rounding-sized step left
// is at the root; the block is that set.  Cost: (passes) x (window) powf pairs per row, so this
// serves short rows; longer ones go to the block-per-row solver of tk_thr.cu.
__device__ __forceinline__ void solve_row_newton(const float* sk, int n, int k, const Math& M, const Problem& P,
                                                 RowSol& R, int& flags) {
  auto key = [&](int i) -> float { return sk[i]; };
  const float c = key(k - 1);
  const float lam = P.lam;
  const bool has_block = (k < n) && (c - lam < key(k));
  const float piv = c;
  int a0 = k, b0 = k;
  float u = 0.0f;
  if (has_block) {
    // window ranks [wl, wh): keys strictly between c - lambda and c + lambda
    int wl = k - 1, wh = k + 1;
    while (wl > 0 && key(wl - 1) - piv < lam) --wl;
    while (wh < n && key(wh) - piv > -lam) ++wh;
    float lo = -lam, hi = key(k) - piv;            // offsets with F >= 0 at lo, F <= 0 at hi
    float off = 0.5f * (lo + hi);
    int prev_ct = -1, prev_cm = -1;
    bool done = false;
#pragma unroll 1
    for (int it = 0; it < 64 && !done; ++it) {
      int ct = wl, cm = 0;                          // ranks above the window are capped whatever gamma is
      float s1 = 0.f, s2 = 0.f;
      for (int i = wl; i < wh; ++i) {
        const float tt = (key(i) - piv) - off;
        const bool top = tt >= lam;
        const bool mid = tt > 0.0f && !top;
        ct += top; cm += mid;
        if (mid) { s1 += M.rho(tt); s2 += M.drho(tt); }
      }
      const int m = k - ct;
      const float Fv = (float)(ct - k) + s1;
      float du = 0.0f;
      bool have = false;
      if (cm > 0 && m >= 1 && s2 > 0.0f) {
        du = (s1 - (float)m) / s2;
        have = true;
        if (ct == prev_ct && cm == prev_cm && fabsf(du) <= 1e-6f * lam) { a0 = ct; b0 = ct + cm; off += du; done = true; }
      }
      if (!done) {
        if (Fv > 0.0f) lo = fmaxf(lo, off); else hi = fminf(hi, off);
        const float cand = off + du;
        const bool inside = have && cand > lo && cand < hi && (it & 7) != 7;
        prev_ct = inside ? ct : -1; prev_cm = inside ? cm : -1;
        const float next = inside ? cand : 0.5f * (lo + hi);
        if (next == off || !(hi > lo)) { a0 = ct; b0 = ct + cm; if (have) off += du; done = true; }
        else off = next;
      }
    }
    if (!done) flags |= TK_FLAG_NOT_CONVERGED;
    u = off;
    if (b0 > a0) u = settle_offset(M, piv, u, a0, b0, n, key);
    else { a0 = k; b0 = k; }
  }
  const bool block = b0 > a0;
  R.piv = piv; R.u = block ? u : 0.0f; R.c = c; R.a0 = a0; R.b0 = b0; R.has_block = block ? 1 : 0;
}

// The same growth by a whole warp for one row (rows of more than 128 elements have a warp to
// themselves): 32 candidates per step.  Lane i tests rank b + i (or a - 1 - i) against the block
// with the i candidates before it already pooled -- its power sums are the block's plus an
// exclusive prefix over the lanes -- which is exactly the test the one-at-a-time loop would make
// when it got there, and the candidates that join are the leading run of passing lanes.  A side
// is left at its first failing candidate, as in the serial loop, so the result is the same; a
// block of m ranks costs about m/32 + 3 steps.  Block sums for the value are then taken in fp64
// by the warp.
template <bool Q4, bool MAG>
__device__ __forceinline__ void solve_row_coop(const float* sk, int n, int k, const Math& M, const Problem& P,
                                               int lane, RowSol& R) {
  auto key = [&](int i) -> float { return sk[i]; };
  const float c = key(k - 1);
  const float vtop_c = M.vtop(c);
  const bool has_block = (k < n) && (vtop_c < key(k));
  const float piv = (MAG && vtop_c < 0.5f * c) ? 0.0f : c;   // as in solve_row_walk
  int a0 = k, b0 = k;
  float u = 0.0f;
  if (has_block) {                                           // uniform over the warp
    const float il3 = P.inv_lam * P.inv_lam * P.inv_lam;
    const float dk = key(k) - piv, dc = c - piv;
    float D1 = dc + dk, D2 = 0.f, D3 = 0.f;
    if (Q4) { D2 = dc * dc + dk * dk; D3 = dc * dc * dc + dk * dk * dk; }
    a0 = k - 1; b0 = k + 1;
    auto excl = [&](float v) -> float {                      // exclusive prefix over the lanes
      float inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const float up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
      return inc - v;
    };
    int below = 1, fails = 0;
    while (fails < 2) {
      const int j = below ? b0 + lane : a0 - 1 - lane;
      const bool valid = below ? (j < n) : (j >= 0);
      const float s = valid ? key(j) : 0.0f;
      const float d = valid ? s - piv : 0.0f;
      float d2 = 0.f, d3 = 0.f, x2 = 0.f, x3 = 0.f;
      const float x1 = excl(d);
      if (Q4) { d2 = d * d; d3 = d2 * d; x2 = excl(d2); x3 = excl(d3); }
      // the block this candidate is tested against: the current one plus the candidates before it
      const int a = below ? a0 : a0 - lane, b = below ? b0 + lane : b0;
      const float cnt = (float)(b - a), m = (float)(k - a);
      const float uu = below ? d : M.vtop(s) - piv;
      const float S1 = D1 + x1, S2 = D2 + x2, S3 = D3 + x3;
      float Sv;
      if (Q4) Sv = (((-cnt * uu + 3.0f * S1) * uu - 3.0f * S2) * uu + S3) * il3;
      else Sv = (S1 - cnt * uu) * P.inv_lam;
      const float Hv = Sv - (MAG ? m * (piv + uu) : m);
      const bool ok = valid && (below ? (Hv < 0.0f) : (Hv > 0.0f));
      const unsigned bal = __ballot_sync(0xffffffffu, ok);
      const int run = (bal == 0xffffffffu) ? 32 : __ffs(~bal) - 1;      // leading run of joining candidates
      if (run > 0) {
        // pool them: inclusive sums at lane run - 1
        D1 += __shfl_sync(0xffffffffu, x1 + d, run - 1);
        if (Q4) { D2 += __shfl_sync(0xffffffffu, x2 + d2, run - 1); D3 += __shfl_sync(0xffffffffu, x3 + d3, run - 1); }
        if (below) b0 += run; else a0 -= run;
        fails = 0;
      }
      if (run < 32) { ++fails; below ^= 1; }
    }
    // ---- block sums in fp64, then the block value (every lane computes the same)
    double E1 = 0.0, E2 = 0.0, E3 = 0.0;
    for (int i = a0 + lane; i < b0; i += 32) {
      const double dd = (double)(key(i) - piv);
      E1 += dd;
      if (Q4) { const double dd2 = dd * dd; E2 += dd2; E3 = fma(dd2, dd, E3); }
    }
    E1 = warp_sum(E1);
    if (Q4) { E2 = warp_sum(E2); E3 = warp_sum(E3); }
    const double cntd = (double)(b0 - a0);
    const double mud = E1 / cntd;
    float M2 = 0.f, M3 = 0.f;
    if (Q4) {
      M2 = (float)(E2 - E1 * mud);
      M3 = (float)(E3 - 3.0 * mud * E2 + 2.0 * mud * mud * E1);
    }
    u = block_value<Q4, MAG>(P.lam, P.lam3, piv, (float)cntd, (float)(k - a0), (float)mud, M2, M3);
    u = settle_offset(M, piv, u, a0, b0, n, key);
  }
  R.piv = piv; R.u = u; R.c = c; R.a0 = a0; R.b0 = b0; R.has_block = has_block ? 1 : 0;
}

// Ranks that can be pooled at all: keys strictly between vtop(c) and c + width(c), c the k-th
// largest key (two binary searches on the sorted row).  An upper bound of the block's size, used
// to choose between the one-lane growth (cheap per member, serial) and the warp's (32 at a time).
__device__ __forceinline__ int window_ranks(const float* sk, int n, int k, const Math& M) {
  const float c = sk[k - 1];
  const float lo_key = M.vtop(c), hi_key = c + M.width(c);
  if (!(k < n) || !(lo_key < sk[k])) return 0;
  int l = 0, r = k;                              // first rank with key < hi_key
  while (l < r) { const int mid = (l + r) >> 1; if (sk[mid] >= hi_key) l = mid + 1; else r = mid; }
  const int wl = l;
  l = k; r = n;                                  // first rank with key <= lo_key
  while (l < r) { const int mid = (l + r) >> 1; if (sk[mid] > lo_key) l = mid + 1; else r = mid; }
  return l - wl;
}

constexpr int kSerialGrowthMax = 224;   // window above which a warp per row grows the block cooperatively

constexpr int kRowsThreads = 128;

// B batches of 32/G rows per warp.  The most batches (32 rows per warp, 16 for n > 64, 8 for
// n > 128) cost the fewest instructions per row; fewer batches give a small problem enough warps
// to fill the machine.
template <int G, int E, int B>
struct RowsGeom {
  static constexpr int N = E * G;                          // padded row length
  static constexpr int RPB = 32 / G;                       // rows per batch
  static constexpr int R = RPB * B;                        // rows per warp
  static constexpr int STRIDE = N | 1;                     // odd: lane r walking row r meets no bank conflict
};

// QM: 0 for q = 2, 1 for q = 4, 2 for any other q (short rows, mask and top-k modes)
// Resident blocks asked of the compiler: 6 with 8 or 16 keys per lane (16 keys: 76 registers instead
// of 82, no spills, and n = 300..512 runs 6 % faster than at 5 blocks; 8 keys: 8 blocks of half the
// batches were measured 3-17 % slower), 3 with 32.
template <int G, int E, int B, int QM, bool MAG>
__global__ void __launch_bounds__(kRowsThreads, E <= 16 ? 6 : 3) tk_rows_kernel(const Problem P) {
  constexpr bool Q4 = QM == 1, GEN = QM == 2;
  constexpr int RPB = RowsGeom<G, E, B>::RPB, R = RowsGeom<G, E, B>::R, BATCHES = B;
  constexpr int STRIDE = RowsGeom<G, E, B>::STRIDE;
  constexpr int WARPS = kRowsThreads / 32;
  __shared__ float sm[WARPS][R][STRIDE];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gw = lane / G, lig = lane % G;        // the lane's row within a batch, its place in the row
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << (gw * G);
  const long long row0 = ((long long)blockIdx.x * WARPS + warp) * R;
  const int n = P.n, k = P.k;
  Math M = make_math(P);
  M.q4 = Q4; M.mag = MAG; M.gen = GEN;      // compile-time constants from here on
  int flags = 0;

  // elements 4 h .. 4 h + 3 of the lane's E consecutive elements of a row (zeros past the row's end)
  auto load4 = [&](const float* base, bool live, int h, float (&v4)[4]) {
    const int e0 = E * lig + 4 * h;
    if (P.vec4) {
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (live && e0 < n) q = __ldg(reinterpret_cast<const float4*>(base) + (e0 >> 2));
      v4[0] = q.x; v4[1] = q.y; v4[2] = q.z; v4[3] = q.w;
    } else {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) v4[c4] = (live && e0 + c4 < n) ? __ldg(base + e0 + c4) : 0.0f;
    }
  };

  // ---- phase 1: sort the keys of every row, batch by batch
  constexpr bool KEEPX = B == 1 && E <= 16;      // a single batch keeps its row in registers for phase 3
  float xkeep[KEEPX ? E : 1];
#pragma unroll 1
  for (int b = 0; b < BATCHES; ++b) {
    const int rr = b * RPB + gw;
    const long long row = row0 + rr;
    const bool live = row < P.rows;
    float s[E];
    bool bad = false;
#pragma unroll
    for (int h = 0; h < E / 4; ++h) {
      float x4[4];
      load4(P.theta + (live ? row : 0) * (long long)n, live, h, x4);
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        const int i = 4 * h + c4;
        const bool in = E * lig + i < n;
        if (in && !isfinite(x4[c4])) bad = true;
        s[i] = in ? sort_key(x4[c4], MAG) : -INFINITY;   // slots past the row sort last
        if (KEEPX) xkeep[KEEPX ? i : 0] = x4[c4];
      }
    }
    if (bad && live) flags |= TK_FLAG_NONFINITE;
    group_sort_keys<G, E>(s, lig, mask);
    float* sk = sm[warp][rr];
#pragma unroll
    for (int i = 0; i < E; ++i) sk[E * lig + i] = s[i];   // rank E lig + i
  }
  __syncwarp();

  // ---- phase 2: lane r solves row r
  RowSol mine;
  mine.piv = 0.f; mine.u = 0.f; mine.c = 0.f; mine.a0 = k; mine.b0 = k; mine.has_block = 0;
  bool coop = false;
  if (G == 32 && E >= 16 && !GEN) {              // rows of more than 256 elements: blocks can be large
    int w = 0;
    if (lane < R && row0 + lane < P.rows) w = window_ranks(sm[warp][lane % R], n, k, M);
    coop = __any_sync(0xffffffffu, w > kSerialGrowthMax);
  }
  if (coop) {
    // the warp grows its rows one after the other, 32 candidates at a time
#pragma unroll 1
    for (int r = 0; r < R; ++r) {
      if (row0 + r < P.rows) {                   // uniform over the warp
        RowSol sol;
        solve_row_coop<Q4, MAG>(sm[warp][r], n, k, M, P, lane, sol);
        if (lane == r) mine = sol;
      }
    }
  } else if (lane < R && row0 + lane < P.rows) {
    if (GEN) solve_row_newton(sm[warp][lane % R], n, k, M, P, mine, flags);
    else solve_row_walk<Q4, MAG>(sm[warp][lane % R], n, k, M, P, mine);
  }
  if (lane < R && row0 + lane < P.rows && P.state_out) {
    tk_rowstate st;
    st.pivot = mine.has_block ? mine.piv : mine.c; st.offset = mine.u; st.a = mine.a0; st.b = mine.b0;
    P.state_out[row0 + lane] = st;
  }
  __syncwarp();

  // ---- phase 3: results by value, in the original order, four elements at a time.  A launch with
  // a single batch of up to 16 keys per lane still has the row in registers; otherwise the row is
  // read again (L1 / L2).
#pragma unroll 1
  for (int b = 0; b < BATCHES; ++b) {
    const int rr = b * RPB + gw;
    const long long row = row0 + rr;
    const bool live = row < P.rows;
    const bool has_block = __shfl_sync(0xffffffffu, mine.has_block, rr) != 0;
    const float piv = __shfl_sync(0xffffffffu, mine.piv, rr);
    const float u = __shfl_sync(0xffffffffu, mine.u, rr);
    const float c = __shfl_sync(0xffffffffu, mine.c, rr);
    const int a0 = __shfl_sync(0xffffffffu, mine.a0, rr);
    const float* x_row = P.theta + (live ? row : 0) * (long long)n;
    float* o_row = P.out + (live ? row : 0) * (long long)n;
    const float wid = has_block ? M.width(piv + u) : 0.0f;
    // class of a key: 2 capped (top singleton), 1 pooled, 0 zero; tt = key - gamma, clamped
    auto classify = [&](float key, float& tt) -> int {
      if (!has_block) { tt = 0.0f; return key >= c ? 2 : 0; }
      const float t = (key - piv) - u;
      tt = fminf(fmaxf(t, 0.0f), wid);
      return t >= wid ? 2 : (t > 0.0f ? 1 : 0);
    };
    auto chi_of = [&](float xv) -> float {
      return MAG ? (signbit(xv) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? xv : 1.0f);
    };
    // up to 16 keys per lane: the lane's part of the row (and of the cotangent) is loaded at once
    // and held; with 32 it is fetched chunk by chunk in every pass
    constexpr bool HOLD = E <= 16;
    float xall[HOLD ? E : 1], gall[HOLD ? E : 1];
    if (HOLD) {
#pragma unroll
      for (int h = 0; h < E / 4; ++h) {
        float v4[4];
        if (KEEPX) {
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) v4[c4] = xkeep[KEEPX ? 4 * h + c4 : 0];
        } else {
          load4(x_row, live, h, v4);
        }
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) xall[HOLD ? 4 * h + c4 : 0] = v4[c4];
      }
      if (P.what != W_FWD) {
#pragma unroll
        for (int h = 0; h < E / 4; ++h) {
          float v4[4];
          load4(P.gout + (live ? row : 0) * (long long)n, live, h, v4);
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) gall[HOLD ? 4 * h + c4 : 0] = v4[c4];
        }
      }
    }
    auto x4_of = [&](int h, float (&v4)[4]) {
      if (HOLD) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) v4[c4] = xall[HOLD ? 4 * h + c4 : 0];
      } else {
        load4(x_row, live, h, v4);
      }
    };
    auto g4_of = [&](const float* g_row, int h, float (&v4)[4]) {
      if (HOLD) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) v4[c4] = gall[HOLD ? 4 * h + c4 : 0];
      } else {
        load4(g_row, live, h, v4);
      }
    };
    auto store4 = [&](int h, const float (&o4)[4]) {
      const int e0 = E * lig + 4 * h;
      if (P.vec4) {
        if (live && e0 < n) reinterpret_cast<float4*>(o_row)[e0 >> 2] = make_float4(o4[0], o4[1], o4[2], o4[3]);
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) if (live && e0 + c4 < n) o_row[e0 + c4] = o4[c4];
      }
    };
    if (P.what == W_FWD) {
#pragma unroll
      for (int h = 0; h < E / 4; ++h) {
        float x4[4], o4[4];
        x4_of(h, x4);
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          float tt;
          const float key = sort_key(x4[c4], MAG);
          const int cls = classify(key, tt);
          float v = cls == 2 ? (MAG ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
          if (MAG) v = signbit(x4[c4]) ? -v : v;
          if (P.mode == TK_TOPK) v *= x4[c4];
          o4[c4] = v;
        }
        store4(h, o4);
      }
    } else {
      // ---- VJP (Prop. 7): o_j = rho'_j (chi_j g_j - A/D) on the pooled block, by value
      const float* g_row = P.gout + (live ? row : 0) * (long long)n;
      float A = 0.f, D = 0.f;
      if (has_block) {
#pragma unroll
        for (int h = 0; h < E / 4; ++h) {
          float x4[4], g4[4];
          x4_of(h, x4);
          g4_of(g_row, h, g4);
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            float tt;
            if (E * lig + 4 * h + c4 < n && classify(sort_key(x4[c4], MAG), tt) == 1) {
              const float dr = M.drho(tt);
              D += dr; A += dr * chi_of(x4[c4]) * g4[c4];
            }
          }
        }
      }
      A = group_sum<G, float>(A, mask);
      D = group_sum<G, float>(D, mask);
      if (MAG && has_block) D += (float)(k - a0);
      const float ratio = D > 0.0f ? A / D : 0.0f;
      // second pass: residuals about the fp32 mean (one fma each, no cancellation) restore what
      // the division rounded away; rho' can be 3/lambda, and an ulp of the mean times that shows
      float A2 = 0.f;
      if (has_block) {
#pragma unroll
        for (int h = 0; h < E / 4; ++h) {
          float x4[4], g4[4];
          x4_of(h, x4);
          g4_of(g_row, h, g4);
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            float tt;
            if (E * lig + 4 * h + c4 < n && classify(sort_key(x4[c4], MAG), tt) == 1)
              A2 += M.drho(tt) * fmaf(chi_of(x4[c4]), g4[c4], -ratio);
          }
        }
      }
      A2 = group_sum<G, float>(A2, mask);
      if (MAG && has_block) A2 -= (float)(k - a0) * ratio;
      const float delta = D > 0.0f ? A2 / D : 0.0f;
#pragma unroll
      for (int h = 0; h < E / 4; ++h) {
        float x4[4], g4[4], o4[4];
        x4_of(h, x4);
        g4_of(g_row, h, g4);
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          float tt;
          const float key = sort_key(x4[c4], MAG);
          const int cls = classify(key, tt);
          const float sgn = (MAG && signbit(x4[c4])) ? -1.0f : 1.0f;
          const float chi = chi_of(x4[c4]);
          float v = 0.0f;
          if (cls == 1) v = M.drho(tt) * (fmaf(chi, g4[c4], -ratio) - delta);
          else if (cls == 2 && MAG) v = chi * g4[c4] * M.top_slope(key);
          v *= sgn;
          if (P.mode == TK_TOPK) v += g4[c4] * (cls == 2 ? 1.0f : (cls == 1 ? M.rho(tt) : 0.0f));
          o4[c4] = v;
        }
        store4(h, o4);
      }
    }
  }
  if (flags && P.status) atomicOr(P.status, flags);
}

template <int G, int E, int B>
cudaError_t launch_rows_gb(const Problem& P, cudaStream_t stream) {
  const long long per_block = (long long)(kRowsThreads / 32) * RowsGeom<G, E, B>::R;
  const unsigned blocks = (unsigned)((P.rows + per_block - 1) / per_block);
  const bool mag = P.mode == TK_TOPKMAG;
  if (P.qm1 > 0.0f) {                          // any other q: rows of up to 128 elements, not the magnitude mode
    if constexpr (G <= 16 && E <= 16) {
      if (mag) return cudaErrorInvalidValue;
      tk_rows_kernel<G, E, B, 2, false><<<blocks, kRowsThreads, 0, stream>>>(P);
      return cudaGetLastError();
    } else {
      return cudaErrorInvalidValue;
    }
  }
  if (P.q4) {
    if (mag) tk_rows_kernel<G, E, B, 1, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, E, B, 1, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  } else {
    if (mag) tk_rows_kernel<G, E, B, 0, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, E, B, 0, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  }
  return cudaGetLastError();
}

// warps below which a launch leaves SMs short of work: 24 per SM
inline long long warps_to_fill() { return (long long)sm_count() * 24; }

// 8 keys per lane.  The most batches per warp that still leave warps_to_fill() warps, out of {1, 2, BMAX}.
template <int G, int BMAX>
cudaError_t launch_rows_g(const Problem& P, cudaStream_t stream) {
  constexpr int RPB = 32 / G;
  if (BMAX > 2 && P.rows / (RPB * BMAX) >= warps_to_fill()) return launch_rows_gb<G, 8, BMAX>(P, stream);
  if (BMAX >= 2 && P.rows / (RPB * 2) >= warps_to_fill()) return launch_rows_gb<G, 8, (BMAX >= 2 ? 2 : 1)>(P, stream);
  return launch_rows_gb<G, 8, 1>(P, stream);
}

}  // namespace

// Forward pass or recomputing VJP for rows of up to 1024 elements when no permutation is asked for.
cudaError_t launch_rows(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  if (P.n > 8 && P.n <= 16) {                  // one lane per row, 16 keys: the whole sort in registers
    P.N = 16;
    return launch_rows_gb<1, 16, 1>(P, stream);
  }
  if (P.n > 512) {                             // one warp per row, 32 keys per lane, up to 2 rows per warp
    P.N = 1024;
    if (P.rows / 2 >= warps_to_fill()) return launch_rows_gb<32, 32, 2>(P, stream);
    return launch_rows_gb<32, 32, 1>(P, stream);
  }
  if (P.n > 256) {                             // one warp per row, 16 keys per lane, up to 4 rows per warp
    P.N = 512;
    if (P.rows / 4 >= warps_to_fill()) return launch_rows_gb<32, 16, 4>(P, stream);
    if (P.rows / 2 >= warps_to_fill()) return launch_rows_gb<32, 16, 2>(P, stream);
    return launch_rows_gb<32, 16, 1>(P, stream);
  }
  int G = 1;
  while (G * 8 < P.n) G <<= 1;
  P.N = G * 8;
  switch (G) {
    case 1: return launch_rows_g<1, 1>(P, stream);
    case 4: return launch_rows_g<4, 4>(P, stream);
    case 8: return launch_rows_g<8, 8>(P, stream);
    case 16: return launch_rows_g<16, 8>(P, stream);
    default: return launch_rows_g<32, 8>(P, stream);
  }
}

}  // namespace tk
