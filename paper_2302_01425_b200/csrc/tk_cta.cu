// tk_cta.cu -- one thread block per row, the whole row resident on chip.
//
// Steps (Sec. 5 of the paper, Prop. 5/6 reduction):
//   load row -> (key, index) packed in 64 bits -> block-wide merge sort in
//   shared memory (stable: ties by ascending index) -> exact isotonic solve
//   -> dual map y = rho(s - v) -> scatter through shared memory -> coalesced
//   store.  Used when the caller wants the permutation (perm_out, tk_argsort);
//   the default forward pass and every VJP sort the keys alone (tk_ctav.cu).
//
// Isotonic solve.  With w = 1_k the singleton minimisers are non-increasing on
// ranks < k and on ranks >= k, so pooling adjacent violators can only ever grow
// ONE block [a, b) around rank k.  Its value gamma is the root of a monotone
// function F; "rank j lies above gamma" is F(s_j) < 0 and "rank j stays a top
// singleton" is F(vtop(s_j)) <= 0, both monotone in j, so a and b are found by
// a block-wide T-ary search, each probe costing O(1) through prefix sums of
// d, d^2, d^3 (d = s - pivot) over the window of ranks that can be pooled.
#include "tk_common.cuh"
#include "tk_cta_sort.cuh"
#include "tk_block_util.cuh"

namespace tk {

namespace {

struct RowSolve {       // per-row scalars shared by all threads
  int a0, b0;           // pooled block [a0, b0) in sorted ranks; a0 == b0 == k: none
  float c, u;           // pivot and gamma - pivot
};

template <int E, int MAXT>
__global__ void __launch_bounds__(MAXT, MAXT == 512 ? 2 : 1)
tk_cta_kernel(const Problem P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int T = blockDim.x;
  const int t = threadIdx.x;
  const int n = P.n, k = P.k, N = P.N;
  const long long row = blockIdx.x;
  const Math M = make_math_q24(P);
  const bool mag = M.mag;

  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);   // pad(N) slots
  float* stage = reinterpret_cast<float*>(smem_raw);                             // aliases keys, [N]
  const int key_slots = pad(N) + 1;
  double* cps = reinterpret_cast<double*>(keys + key_slots);                     // 3 x (T + 1)
  double* redd = cps + 3 * (T + 1);                                              // 40 doubles
  int* redi = reinterpret_cast<int*>(redd + 40);                                 // 40 ints
  __shared__ RowSolve sol;
  __shared__ int row_flags;

  if (t == 0) row_flags = 0;

  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[E];
  bool bad = false;

  cta_load_sort<E>(P, x_row, keys, r, bad);
  // thread t now holds sorted ranks [tE, tE + E) in r[], and keys[] holds them all

  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
    for (int i = t; i < n; i += T) pr[i] = un_idx(keys[pad(i)]);
  }
  if (P.sorted_out) {
    float* so = P.sorted_out + row * (long long)n;
    for (int i = t; i < n; i += T) so[i] = un_key(keys[pad(i)]);
  }
  if (P.what == W_ARGSORT) {
    if (bad && P.status) atomicOr(P.status, TK_FLAG_NONFINITE);
    return;
  }

  // ---- isotonic solve
  const float c = un_key(keys[pad(k - 1)]);
  const float vtop_c = M.vtop(c);
  bool has_block = false;
  if (k < n) {
    float sk = un_key(keys[pad(k)]);
    has_block = vtop_c < sk;
  }
  // Pivot for the arithmetic around the pooled block.  The block's keys lie in
  // (vtop(c), c + width(c)); when that window stays within a factor two of c the
  // pivot c makes every difference below exact.  For phi even and large lambda the
  // window reaches far below c (gamma << c); then the keys themselves are the
  // well-scaled quantity and the pivot is 0.
  const float piv = (mag && vtop_c < 0.5f * c) ? 0.0f : c;
#define TK_D(i) (un_key(r[i]) - piv)

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
          float di = un_key(keys[pad(i)]) - piv;
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
        float dm = un_key(keys[pad(mid)]) - piv;
        if (dm >= x) L = mid + 1; else R = mid;
      }
      return L;
    };
    auto count_gt = [&](float x, int L, int R) -> int {
      while (L < R) {
        int mid = (L + R) >> 1;
        float dm = un_key(keys[pad(mid)]) - piv;
        if (dm > x) L = mid + 1; else R = mid;
      }
      return L;
    };
    // predB(j): rank j lies strictly above gamma.  predA(j): rank j stays a top singleton.
    auto predB = [&](int j) -> bool {
      if (j < k) return true;
      if (j >= wh) return false;
      float tau = un_key(keys[pad(j)]);
      float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      int r_hi = count_ge(uu + M.width(tau), wl, k);
      return evalF(uu, r_hi, j) < 0.0f;
    };
    auto predA = [&](int j) -> bool {
      if (j < wl) return true;
      if (j >= k) return false;
      float tau = M.vtop(un_key(keys[pad(j)]));
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
      sol.u = settle_offset(M, piv, (float)uu, a0, b0, n, [&](int i) -> float { return un_key(keys[pad(i)]); });
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

  // ---- dual map in sorted coordinates: y^s = rho(s - v)
  const float wid = has_block ? M.width(piv + u) : 0.0f;
  auto y_of = [&](int rk, unsigned long long e) -> float {
    if (rk < a0) return mag ? M.vtop(un_key(e)) : 1.0f;    // top singleton: rho(s - vtop) = phi'(vtop)
    if (rk < b0) return M.rho(fminf(fmaxf((un_key(e) - piv) - u, 0.0f), wid));
    return 0.0f;
  };
  __syncthreads();       // every read of keys[] is done; stage[] may overwrite it

  {   // forward pass only: tk_vjp never asks for a permutation, so it never comes here
#pragma unroll
    for (int i = 0; i < E; ++i) {
      int idx = un_idx(r[i]);
      if (t * E + i < n && idx < n) {
        float yv = y_of(t * E + i, r[i]);
        stage[idx] = (mag && un_neg(r[i])) ? -yv : yv;
      }
    }
    __syncthreads();
    float* o_row = P.out + row * (long long)n;
    if (P.vec4) {
      const float4* s4 = reinterpret_cast<const float4*>(stage);
      const float4* x4 = reinterpret_cast<const float4*>(x_row);
      float4* o4 = reinterpret_cast<float4*>(o_row);
      for (int v = t; 4 * v < n; v += T) {
        float4 q = s4[v];
        if (P.mode == TK_TOPK) { float4 xx = __ldg(x4 + v); q.x *= xx.x; q.y *= xx.y; q.z *= xx.z; q.w *= xx.w; }
        o4[v] = q;
      }
    } else {
      for (int i = t; i < n; i += T) {
        float q = stage[i];
        if (P.mode == TK_TOPK) q *= __ldg(x_row + i);
        o_row[i] = q;
      }
    }
  }
#undef TK_D
  if (t == 0 && row_flags && P.status) atomicOr(P.status, row_flags);
}

}  // namespace

size_t cta_smem_bytes(int N, int T) {
  size_t keys = (size_t)(N + (N >> PAD_SHIFT) + 1) * 8;
  return keys + (size_t)3 * (T + 1) * 8 + 40 * 8 + 40 * 4 + 64;
}

// Picks items-per-thread for a padded row length.
// Items per thread.  The merge rounds are latency-bound, so the choice favours resident warps:
// 8 items from N = 512 (64-thread blocks, many per SM), 16 from N = 4096 with registers capped at 64.
static int pick_items(int N) { return N >= 4096 ? 16 : (N >= 512 ? 8 : 4); }

int cta_padded_length(int n) {
  int N = 128;
  while (N < n) N <<= 1;
  return N;
}

cudaError_t launch_cta(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  P.N = cta_padded_length(P.n);
  const int E = pick_items(P.N);
  const int T = P.N / E;
  const size_t smem = cta_smem_bytes(P.N, T);
  cudaError_t err;
  void (*kern)(const Problem) = nullptr;
  switch (E) {
    case 4: kern = tk_cta_kernel<4, 128>; break;
    case 8: kern = tk_cta_kernel<8, 512>; break;
    default: kern = (T > 512) ? tk_cta_kernel<16, 1024> : tk_cta_kernel<16, 512>; break;
  }
  // The opt-in to large dynamic shared memory is per function and per device; it is raised
  // once to the largest size this file ever asks for.
  static bool configured[4][64] = {};
  int dev = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  const int slot = (E == 4) ? 0 : (E == 8) ? 1 : (T > 512 ? 3 : 2);
  if (dev < 0 || dev >= 64 || !configured[slot][dev]) {
    const int max_smem = (int)cta_smem_bytes(16384, 1024);
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) configured[slot][dev] = true;
  }
  dim3 grid((unsigned)P.rows), block((unsigned)T);
  kern<<<grid, block, smem, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace tk
