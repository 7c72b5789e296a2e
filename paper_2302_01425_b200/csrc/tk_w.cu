// tk_w.cu -- the relaxed operator for any sorted w (Sec. 3: LP forms of sort and rank over the
// permutahedron P(w); Sec. 4 with phi(x) = x):
//   y_R(x, w) = argmax_{y in P(w)} <x, y> - R(y) = grad R*(x - u*),  u* = v*_{sigma^-1},
//   v* = argmin_{v_1 >= .. >= v_n} sum_i r*(s_i - v_i) + w_i v_i                     (Prop. 5),
// and its VJP in x (Prop. 7).  With w = 1_k this is the relaxed top-k mask, which the other kernels
// solve through its single pooled block; a general w pools many blocks, so this one runs pool-
// adjacent-violators itself, in parallel:
//   1. the row is sorted (descending, ties by index) as 64-bit (key, index) words in shared memory
//      (bitonic network);
//   2. prefix sums of the sorted keys (about a pivot, in fp64) and of w make the value of ANY
//      candidate block [lo, hi) an O(1) computation: gamma = (sum s - lambda sum w) / N for p = 2,
//      the root of N g^3 - 3 S1 g^2 + 3 S2 g - S3 + lambda^3 sum w = 0 for p = 4/3 (App. A.6);
//   3. rounds over the list of blocks: every block's value is computed, every boundary whose left
//      value is strictly smaller than its right value is erased (a run of such boundaries merges a
//      whole chain at once: the pooled value of two blocks lies between their values, so a chain
//      that violates pairwise still violates after partial merging), until no boundary violates.
//      Pooling a violating pair is always part of the solution (App. B.2), so the order of the
//      merges does not matter and the result is the partition sequential PAV ends with;
//   4. y^s_i = rho(s_i - gamma_B(i)) goes back through the permutation; for the VJP the block sums
//      D_B = sum rho', A_B = sum rho' g^s come from two more prefix sums.
// One thread block per row, rows of up to 2048 elements.
#include "tk_common.cuh"

namespace tk {

namespace {

constexpr int kWThreads = 256;
constexpr int kWMaxN = 2048;

// exclusive block-wide prefix sum of one double per thread (in place); returns the total
__device__ __forceinline__ double w_block_exscan(double v, double* sh_warp, double* total) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  __syncthreads();
  if (lane == 31) sh_warp[warp] = inc;
  __syncthreads();
  double base = 0.0, tot = 0.0;
#pragma unroll
  for (int wv = 0; wv < kWThreads / 32; ++wv) {
    const double s = sh_warp[wv];
    if (wv < warp) base += s;
    tot += s;
  }
  *total = tot;
  return base + inc - v;
}

// Root of f(g) = N g^3 + 3 M2 g + c (M2 >= 0: increasing), the block's cubic about its own mean.
__device__ __forceinline__ double w_cubic_root(double N, double M2, double c) {
  if (c == 0.0) return 0.0;
  // |root| <= cbrt(|c| / N); safeguarded Newton inside [lo, hi]
  const double r0 = cbrt(fabs(c) / N);
  double lo = c > 0.0 ? -r0 : 0.0, hi = c > 0.0 ? 0.0 : r0;
  double g = M2 > 0.0 ? fmin(fmax(-c / (3.0 * M2), lo), hi) : (c > 0.0 ? -r0 : r0);
#pragma unroll 1
  for (int it = 0; it < 80; ++it) {
    const double f = (N * g * g + 3.0 * M2) * g + c;
    if (f > 0.0) hi = g; else lo = g;
    const double fp = 3.0 * (N * g * g + M2);
    double nx = fp > 0.0 ? g - f / fp : 0.5 * (lo + hi);
    if (!(nx > lo && nx < hi)) nx = 0.5 * (lo + hi);
    if (fabs(nx - g) <= 1e-15 * (fabs(nx) + r0)) { g = nx; break; }
    g = nx;
  }
  return g;
}

struct WArrays {
  unsigned long long* keys;   // [N] packed (key, index), later reused as float out_s[n]
  float* s;                   // [n] sorted keys
  unsigned short* idx;        // [n] original index of rank i
  double* p1;                 // [n + 1] prefix of d = s - pivot
  double* p2;                 // [n + 1] prefix of d^2   (q = 4)
  double* p3;                 // [n + 1] prefix of d^3   (q = 4)
  double* pw;                 // [n + 1] prefix of w
  int* starts[2];             // block starts, ping-pong
  double* gam;                // [n] value per block (relative to the pivot)
  double* gam2;               // [n] the values carried to the next round's list (NaN: to be computed)
};

template <bool Q4>
__device__ __forceinline__ double w_block_value(const WArrays& A, int lo, int hi, double lam, double lam3) {
  const double N = (double)(hi - lo);
  const double S1 = A.p1[hi] - A.p1[lo], W = A.pw[hi] - A.pw[lo];
  if (!Q4) return (S1 - lam * W) / N;
  if (hi - lo == 1) return S1 - lam * cbrt(W);             // (g - d)^3 + lam^3 w = 0
  const double S2 = A.p2[hi] - A.p2[lo], S3 = A.p3[hi] - A.p3[lo];
  const double mu = S1 / N;
  const double M2 = fmax(S2 - S1 * mu, 0.0);
  const double M3 = S3 - 3.0 * mu * S2 + 2.0 * mu * mu * S1;
  // sum (g - d_i)^3 + lam^3 W = 0 with g = mu + h:  N h^3 + 3 M2 h - M3 + lam^3 W = 0
  return mu + w_cubic_root(N, M2, lam3 * W - M3);
}

// what: W_FWD or W_VJP.  w_rows: 1 (one w for every row) or rows.
template <bool Q4>
__global__ void __launch_bounds__(kWThreads) tk_w_kernel(const Problem P, const float* __restrict__ w_all,
                                                         const int w_shared, const int N) {
  extern __shared__ __align__(16) unsigned char w_smem[];
  __shared__ double sh_warp[kWThreads / 32];
  const int t = threadIdx.x, n = P.n;
  const long long row = blockIdx.x;
  const double lam = (double)P.lam, lam3 = lam * lam * lam;
  // ---- carve the shared memory
  WArrays A;
  unsigned char* ptr = w_smem;
  A.keys = reinterpret_cast<unsigned long long*>(ptr); ptr += (size_t)N * 8;
  A.p1 = reinterpret_cast<double*>(ptr); ptr += (size_t)(n + 1) * 8;
  A.pw = reinterpret_cast<double*>(ptr); ptr += (size_t)(n + 1) * 8;
  A.p2 = reinterpret_cast<double*>(ptr); if (Q4) ptr += (size_t)(n + 1) * 8;
  A.p3 = reinterpret_cast<double*>(ptr); if (Q4) ptr += (size_t)(n + 1) * 8;
  A.gam = reinterpret_cast<double*>(ptr); ptr += (size_t)n * 8;
  A.gam2 = reinterpret_cast<double*>(ptr); ptr += (size_t)n * 8;
  A.s = reinterpret_cast<float*>(ptr); ptr += (size_t)n * 4;
  A.starts[0] = reinterpret_cast<int*>(ptr); ptr += (size_t)(n + 1) * 4;
  A.starts[1] = reinterpret_cast<int*>(ptr); ptr += (size_t)(n + 1) * 4;
  A.idx = reinterpret_cast<unsigned short*>(ptr);

  const float* x_row = P.theta + row * (long long)n;
  const float* w_row = w_all + (w_shared ? 0 : row * (long long)n);
  bool bad = false;
  // ---- 1. sort: larger packed word first; equal keys in ascending index; padding sorts last
  for (int i = t; i < N; i += kWThreads) {
    unsigned long long e = 0ull;
    if (i < n) {
      const float x = TK_IN_BOUNDS(row * (long long)n + i, 1, P.rows * (long long)n, P.status) ? __ldg(x_row + i) : 0.0f;
      bad |= !(fabsf(x) < INFINITY);
      e = ((unsigned long long)f2key(sort_key(x, false)) << 32) | (unsigned)(0xFFFF - i);
      e |= 0x10000ull;                       // a real element outranks the padding (0) even at the smallest key
    }
    A.keys[i] = e;
  }
  __syncthreads();
  for (int kk = 2; kk <= N; kk <<= 1) {
    for (int j = kk >> 1; j > 0; j >>= 1) {
      for (int i = t; i < N; i += kWThreads) {
        const int l = i ^ j;
        if (l > i && TK_IN_BOUNDS(l, 1, N, P.status)) {
          const unsigned long long a = A.keys[i], b = A.keys[l];
          const bool desc = (i & kk) == 0;
          if ((a < b) == desc) { A.keys[i] = b; A.keys[l] = a; }
        }
      }
      __syncthreads();
    }
  }
  for (int i = t; i < n; i += kWThreads) {
    const unsigned long long e = A.keys[i];
    A.s[i] = key2f((uint32_t)(e >> 32));
    A.idx[i] = (unsigned short)(0xFFFF - (int)(e & 0xFFFFu));
    if (!TK_IN_BOUNDS(A.idx[i], 1, n, P.status)) A.idx[i] = 0;
  }
  __syncthreads();
  const double pivot = (double)A.s[n / 2];
  // ---- 2. prefix sums: every thread owns a contiguous chunk
  const int chunk = (n + kWThreads - 1) / kWThreads;
  const int c_lo = min(t * chunk, n), c_hi = min(c_lo + chunk, n);
  {
    double a1 = 0.0, a2 = 0.0, a3 = 0.0, aw = 0.0;
    for (int i = c_lo; i < c_hi; ++i) {
      const double d = (double)A.s[i] - pivot;
      a1 += d; aw += (double)__ldg(w_row + i);
      if (Q4) { a2 += d * d; a3 += d * d * d; }
    }
    double tot;
    double b1 = w_block_exscan(a1, sh_warp, &tot);
    double bw = w_block_exscan(aw, sh_warp, &tot);
    double b2 = 0.0, b3 = 0.0;
    if (Q4) { b2 = w_block_exscan(a2, sh_warp, &tot); b3 = w_block_exscan(a3, sh_warp, &tot); }
    for (int i = c_lo; i < c_hi; ++i) {
      A.p1[i] = b1; A.pw[i] = bw;
      if (Q4) { A.p2[i] = b2; A.p3[i] = b3; }
      const double d = (double)A.s[i] - pivot;
      b1 += d; bw += (double)__ldg(w_row + i);
      if (Q4) { b2 += d * d; b3 += d * d * d; }
    }
    if (c_hi == n && c_lo < n) {
      A.p1[n] = b1; A.pw[n] = bw;
      if (Q4) { A.p2[n] = b2; A.p3[n] = b3; }
    }
    for (int i = t; i <= n; i += kWThreads) A.starts[0][i] = i;
  }
  __syncthreads();
  // ---- 3. rounds of merging.  A block's value is computed when the block is formed and carried from
  // round to round until a merge changes the block (NaN marks a value still to be computed).
  int nb = n, cur = 0;
  double* gam = A.gam;
  double* gnx = A.gam2;
  for (int j = t; j < n; j += kWThreads) gam[j] = nan("");
  __syncthreads();
#pragma unroll 1
  for (int round = 0; round < n; ++round) {
    const int* st = A.starts[cur];
    int* nx = A.starts[cur ^ 1];
    for (int j = t; j < nb; j += kWThreads)
      if (gam[j] != gam[j]) gam[j] = w_block_value<Q4>(A, st[j], j + 1 < nb ? st[j + 1] : n, lam, lam3);
    __syncthreads();
    // keep the start of block j unless block j - 1 violates against it
    const int bchunk = (nb + kWThreads - 1) / kWThreads;
    const int j_lo = min(t * bchunk, nb), j_hi = min(j_lo + bchunk, nb);
    int kept = 0;
    for (int j = j_lo; j < j_hi; ++j) kept += (j == 0) || !(gam[j - 1] < gam[j]);
    double tot;
    int base = (int)w_block_exscan((double)kept, sh_warp, &tot);
    for (int j = j_lo; j < j_hi; ++j)
      if ((j == 0) || !(gam[j - 1] < gam[j])) {
        // block j keeps its value unless it absorbs block j + 1
        const bool grows = j + 1 < nb && gam[j] < gam[j + 1];
        if (TK_IN_BOUNDS(base, 1, n + 1, P.status)) { nx[base] = st[j]; gnx[base] = grows ? nan("") : gam[j]; }
        ++base;
      }
    const int nb2 = (int)tot;
    __syncthreads();
    cur ^= 1;
    { double* tmp = gam; gam = gnx; gnx = tmp; }
    if (nb2 == nb) break;
    nb = nb2;
  }
  // values of the final blocks (all known unless the round cap was hit)
  {
    const int* st = A.starts[cur];
    for (int j = t; j < nb; j += kWThreads)
      if (gam[j] != gam[j]) gam[j] = w_block_value<Q4>(A, st[j], j + 1 < nb ? st[j + 1] : n, lam, lam3);
    if (t == 0 && TK_IN_BOUNDS(nb, 1, n + 1, P.status)) A.starts[cur][nb] = n;
  }
  __syncthreads();
  // ---- 4. results, back through the permutation (out_s reuses the sort buffer)
  const int* st = A.starts[cur];
  float* out_s = reinterpret_cast<float*>(A.keys);
  const float inv_lam = P.inv_lam;
  auto block_of = [&](int i) -> int {          // last block whose start is <= i
    int lo = 0, hi = nb - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (st[mid] <= i) lo = mid; else hi = mid - 1; }
    return lo;
  };
  if (P.what == W_FWD) {
    for (int i = t; i < n; i += kWThreads) {
      const int b = block_of(i);
      const float tt = (float)(((double)A.s[i] - pivot) - gam[b]);
      const float a = tt * inv_lam;
      out_s[A.idx[i]] = Q4 ? a * a * a : a;
    }
  } else {
    // D_B = sum rho', A_B = sum rho' g^s over each block: two more prefix sums (p1, pw are free now)
    const float* g_row = P.gout + row * (long long)n;
    double a1 = 0.0, a2 = 0.0;
    for (int i = c_lo; i < c_hi; ++i) {
      const int b = block_of(i);
      const float tt = (float)(((double)A.s[i] - pivot) - gam[b]);
      const float a = tt * inv_lam;
      const double dr = Q4 ? 3.0 * (double)a * (double)a * (double)inv_lam : (double)inv_lam;
      a1 += dr; a2 += dr * (double)__ldg(g_row + A.idx[i]);
    }
    double tot;
    double b1 = w_block_exscan(a1, sh_warp, &tot);
    double b2 = w_block_exscan(a2, sh_warp, &tot);
    __syncthreads();
    for (int i = c_lo; i < c_hi; ++i) {
      A.p1[i] = b1; A.pw[i] = b2;
      const int b = block_of(i);
      const float tt = (float)(((double)A.s[i] - pivot) - gam[b]);
      const float a = tt * inv_lam;
      const double dr = Q4 ? 3.0 * (double)a * (double)a * (double)inv_lam : (double)inv_lam;
      b1 += dr; b2 += dr * (double)__ldg(g_row + A.idx[i]);
    }
    if (c_hi == n && c_lo < n) { A.p1[n] = b1; A.pw[n] = b2; }
    __syncthreads();
    for (int i = t; i < n; i += kWThreads) {
      const int b = block_of(i);
      const int lo = st[b], hi = TK_IN_BOUNDS(b + 1, 1, n + 1, P.status) ? st[b + 1] : n;
      const double D = A.p1[hi] - A.p1[lo], Ab = A.pw[hi] - A.pw[lo];
      const float tt = (float)(((double)A.s[i] - pivot) - gam[b]);
      const float a = tt * inv_lam;
      const double dr = Q4 ? 3.0 * (double)a * (double)a * (double)inv_lam : (double)inv_lam;
      const double gs = (double)__ldg(g_row + A.idx[i]);
      // a singleton's own mean is its g (the difference of two prefix sums would return rounding noise there)
      const double mean = hi - lo == 1 ? gs : (D > 0.0 ? Ab / D : 0.0);
      out_s[A.idx[i]] = (hi - lo > 1 && D > 0.0) ? (float)(dr * (gs - mean)) : 0.0f;
      // the cotangent pulled back to w, in w's own order: A_B / D_B for every rank of the block (a
      // singleton has y = w: its entry is g also where rho' vanishes)
      if (P.sorted_out && TK_IN_BOUNDS(row * (long long)n + i, 1, P.rows * (long long)n, P.status))
        P.sorted_out[row * (long long)n + i] = (float)mean;
    }
  }
  __syncthreads();
  float* o_row = P.out + row * (long long)n;
  for (int i = t; i < n; i += kWThreads)
    if (TK_IN_BOUNDS(row * (long long)n + i, 1, P.rows * (long long)n, P.status)) o_row[i] = out_s[i];
  if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
}

}  // namespace

int w_max_n() { return kWMaxN; }

// Forward pass (P.what == W_FWD) or VJP (W_VJP, cotangent in P.gout; in theta, and in w when P.sorted_out
// is given) of the relaxed operator over P(w); w: device [w_rows * n], every row non-increasing; w_rows is 1 or P.rows.
cudaError_t launch_w(const Problem& P, const float* w, long long w_rows, cudaStream_t stream) {
  int N = 32;
  while (N < P.n) N <<= 1;
  const bool q4 = P.q4 != 0;
  const size_t smem = (size_t)N * 8 + (size_t)(P.n + 1) * 8 * (q4 ? 4 : 2) + (size_t)P.n * 20 + (size_t)(P.n + 1) * 8 +
                      (size_t)P.n * 2 + 64;
  auto kern = q4 ? tk_w_kernel<true> : tk_w_kernel<false>;
  static bool configured[64][2];
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !configured[dev][q4]) {
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) configured[dev][q4] = true;
  }
  kern<<<(unsigned)P.rows, kWThreads, smem, stream>>>(P, w, w_rows == 1 ? 1 : 0, N);
  return cudaGetLastError();
}

}  // namespace tk
