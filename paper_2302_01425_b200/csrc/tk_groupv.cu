// tk_groupv.cu -- short rows (n <= 512), the default forward pass and VJP: sort of the KEYS only.
//
// Given gamma and the edges of the pooled block, the output (and the VJP) of every element is a
// function of its own key: key >= gamma + width -> capped, gamma < key < gamma + width -> pooled,
// else zero.  So the permutation is never needed to place the results: the row is loaded once,
// its 32-bit keys are sorted by the same network as in tk_group.cu (a compare-exchange is one
// max and one min; half the shuffles of the (key, index) sort), the isotonic solve runs on the
// sorted keys, and each lane then maps ITS OWN original elements by value and stores them where it
// loaded them.  No index, no scatter, no staging buffer.  Equal keys get equal results, so the
// stable order among ties is immaterial here; tk_argsort and perm_out use the (key, index) sort.
//
// Same layout (G lanes x 8 elements, or one warp x 16 elements for 256 < n <= 512) and the same
// solve (Sec. 5; App. A.6) as tk_group.cu.
#include "tk_common.cuh"
#include "tk_group_sort.cuh"
#include "tk_key_sort.cuh"

namespace tk {

namespace {

template <int G, int EPL>
__global__ void __launch_bounds__(128, EPL == 8 ? 8 : 4) tk_groupv_kernel(const Problem P) {
  constexpr int N = G * EPL;
  constexpr int GROUPS = 128 / G;
  constexpr int STRIDE = N + N / EPL + 1;
  __shared__ float sm[GROUPS][4][STRIDE];     // sorted keys, prefix sums of d, d^2, d^3
  auto pad8 = [](int i) -> int { return i + i / EPL; };

  const int tid = threadIdx.x;
  const int grp = tid / G, lig = tid % G;
  const long long row = (long long)blockIdx.x * GROUPS + grp;
  if (row >= P.rows) return;                  // whole groups leave together
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << ((tid & 31) / G * G);
  const int n = P.n, k = P.k;
  const Math M = make_math(P);
  const bool mag = M.mag;
  float* sk = sm[grp][0];
  float* p1 = sm[grp][1];
  float* p2 = sm[grp][2];
  float* p3 = sm[grp][3];

  // ---- load: the lane's 8 consecutive elements; they stay in x[] for the epilogue
  const float* x_row = P.theta + row * (long long)n;
  float x[EPL], s[EPL];
  bool bad = false;
#pragma unroll
  for (int h = 0; h < EPL / 4; ++h) {
    const int base = EPL * lig + 4 * h;
    if (P.vec4) {
      float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
      if (base < n) q = __ldg(reinterpret_cast<const float4*>(x_row) + (base >> 2));
      x[4 * h] = q.x; x[4 * h + 1] = q.y; x[4 * h + 2] = q.z; x[4 * h + 3] = q.w;
    } else {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) x[4 * h + c4] = (base + c4 < n) ? __ldg(x_row + base + c4) : 0.0f;
    }
  }
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const bool in = EPL * lig + i < n;
    if (in && !isfinite(x[i])) bad = true;
    s[i] = in ? sort_key(x[i], mag) : -INFINITY;        // slots past the row sort last
  }
  group_sort_keys<G, EPL>(s, lig, mask);      // lane `lig` holds sorted ranks [EPL lig, EPL lig + EPL)
  int flags = bad ? TK_FLAG_NONFINITE : 0;

#pragma unroll
  for (int i = 0; i < EPL; ++i) sk[pad8(EPL * lig + i)] = s[i];
  __syncwarp(mask);

  // ---- isotonic solve (same derivation as the block-per-row kernel)
  const float c = sk[pad8(k - 1)];
  const float vtop_c = M.vtop(c);
  bool has_block = false;
  if (k < n) has_block = vtop_c < sk[pad8(k)];
  const float piv = (mag && vtop_c < 0.5f * c) ? 0.0f : c;
  int a0 = k, b0 = k;
  float u = 0.0f;
  if (has_block) {
    const float W_hi = (piv == c) ? M.width(c) : c + M.width(c);
    const float W_lo = vtop_c - piv;
    int c_hi = 0, c_lo = 0;
    float s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      const float di = s[i] - piv;
      const bool valid = (EPL * lig + i) < n;
      const bool ge_hi = valid && (di >= W_hi);
      const bool gt_lo = valid && (di > W_lo);
      c_hi += ge_hi; c_lo += gt_lo;
      if (gt_lo && !ge_hi) { s1 += di; float d2 = di * di; s2 += d2; s3 += d2 * di; }
    }
    const int wl = group_sum<G, int>(c_hi, mask);
    const int wh = group_sum<G, int>(c_lo, mask);
    {
      // exclusive prefix sums of the window terms: lane offsets by shuffles, then a second pass
      float o1 = group_excl<G>(s1, lig, mask), o2 = 0.f, o3 = 0.f;
      if (M.q4) { o2 = group_excl<G>(s2, lig, mask); o3 = group_excl<G>(s3, lig, mask); }
#pragma unroll
      for (int i = 0; i < EPL; ++i) {
        const int rk = EPL * lig + i;
        p1[pad8(rk)] = o1;
        if (M.q4) { p2[pad8(rk)] = o2; p3[pad8(rk)] = o3; }
        if (rk >= wl && rk < wh) { const float di = s[i] - piv; o1 += di; const float d2 = di * di; o2 += d2; o3 += d2 * di; }
      }
      if (lig == G - 1) { p1[pad8(N)] = o1; if (M.q4) { p2[pad8(N)] = o2; p3[pad8(N)] = o3; } }
    }
    __syncwarp(mask);

    auto evalF = [&](float uu, int r_hi, int r_lo) -> float {
      const float cnt = (float)(r_lo - r_hi);
      const float D1 = p1[pad8(r_lo)] - p1[pad8(r_hi)];
      float S;
      if (M.q4) {
        const float D2 = p2[pad8(r_lo)] - p2[pad8(r_hi)], D3 = p3[pad8(r_lo)] - p3[pad8(r_hi)];
        S = (((-cnt * uu + 3.0f * D1) * uu - 3.0f * D2) * uu + D3) * (P.inv_lam * P.inv_lam * P.inv_lam);
      } else {
        S = (D1 - cnt * uu) * P.inv_lam;
      }
      if (mag) S = S / (piv + uu);
      return (float)(r_hi - k) + S;
    };
    auto count_ge = [&](float x, int L, int R) -> int {
      while (L < R) { int mid = (L + R) >> 1; if (sk[pad8(mid)] - piv >= x) L = mid + 1; else R = mid; }
      return L;
    };
    auto count_gt = [&](float x, int L, int R) -> int {
      while (L < R) { int mid = (L + R) >> 1; if (sk[pad8(mid)] - piv > x) L = mid + 1; else R = mid; }
      return L;
    };
    auto predB = [&](int j) -> bool {      // rank j lies strictly above gamma
      if (j < k) return true;
      if (j >= wh) return false;
      const float tau = sk[pad8(j)];
      const float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      const int r_hi = count_ge(uu + M.width(tau), wl, k);
      return evalF(uu, r_hi, j) < 0.0f;
    };
    auto predA = [&](int j) -> bool {      // rank j stays a top singleton
      if (j < wl) return true;
      if (j >= k) return false;
      const float tau = M.vtop(sk[pad8(j)]);
      const float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      const int r_lo = count_gt(uu, k, wh);
      return evalF(uu, j, r_lo) <= 0.0f;
    };
    // G-ary search: the chunk (lane) that holds the boundary, then the rank inside it
    int tb = group_sum<G, int>(predB(EPL * lig) ? 1 : 0, mask);
    int ta = group_sum<G, int>(predA(EPL * lig) ? 1 : 0, mask);
    tb = max(tb - 1, 0); ta = max(ta - 1, 0);
    int cb = 0, ca = 0;
    for (int i = lig; i < EPL; i += G) { cb += predB(EPL * tb + i) ? 1 : 0; ca += predA(EPL * ta + i) ? 1 : 0; }
    cb = group_sum<G, int>(cb, mask);
    ca = group_sum<G, int>(ca, mask);
    b0 = min(max(EPL * tb + cb, k + 1), wh);
    a0 = max(min(EPL * ta + ca, k - 1), wl);

    // block sums over [a0, b0), summed directly
    float f1 = 0.f, f2 = 0.f, f3 = 0.f;
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      const int rk = EPL * lig + i;
      if (rk >= a0 && rk < b0) { const float di = s[i] - piv; f1 += di; const float d2 = di * di; f2 += d2; f3 += d2 * di; }
    }
    // at most 512 well-scaled terms: fp32 tree sums are accurate to a few ulp
    const double D1 = (double)group_sum<G, float>(f1, mask);
    double D2 = 0.0, D3 = 0.0;
    if (M.q4) { D2 = (double)group_sum<G, float>(f2, mask); D3 = (double)group_sum<G, float>(f3, mask); }
    const double cnt = (double)(b0 - a0), m = (double)(k - a0);
    const double u_left = mag ? (double)W_lo : D1 / cnt - (double)P.lam * (double)cbrtf((float)(m / cnt)) * 1.000001;
    int nc = 0;
    u = (float)solve_block_u(M.q4, mag, (double)P.lam, (double)piv, cnt, m, D1, D2, D3, u_left, &nc);
    u = settle_offset(M, piv, u, a0, b0, n, [&](int i) -> float { return sk[pad8(i)]; });
    if (nc) flags |= TK_FLAG_NOT_CONVERGED;
  }
  if (P.state_out && lig == 0) {
    tk_rowstate st;
    st.pivot = has_block ? piv : c; st.offset = u; st.a = a0; st.b = b0;
    P.state_out[row] = st;
  }


  // ---- epilogue by value, in the original order
  const float wid = has_block ? M.width(piv + u) : 0.0f;
  // class of a key: 2 capped (top singleton), 1 pooled, 0 zero; tt = key - gamma, clamped
  auto classify = [&](float key, float& tt) -> int {
    if (!has_block) { tt = 0.0f; return key >= c ? 2 : 0; }
    const float t = (key - piv) - u;
    tt = fminf(fmaxf(t, 0.0f), wid);
    return t >= wid ? 2 : (t > 0.0f ? 1 : 0);
  };
  float o[EPL];
  if (P.what == W_FWD) {
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      float tt;
      const float key = sort_key(x[i], mag);
      const int cls = classify(key, tt);
      float v = cls == 2 ? (mag ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
      if (mag) v = signbit(x[i]) ? -v : v;
      if (P.mode == TK_TOPK) v *= x[i];
      o[i] = v;
    }
  } else {
    // ---- VJP (Prop. 7): o_j = rho'_j (chi_j g_j - A/D) on the pooled block, by value
    const float* g_row = P.gout + row * (long long)n;
    float g[EPL];
#pragma unroll
    for (int h = 0; h < EPL / 4; ++h) {
      const int base = EPL * lig + 4 * h;
      if (P.vec4) {
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        if (base < n) q = __ldg(reinterpret_cast<const float4*>(g_row) + (base >> 2));
        g[4 * h] = q.x; g[4 * h + 1] = q.y; g[4 * h + 2] = q.z; g[4 * h + 3] = q.w;
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) g[4 * h + c4] = (base + c4 < n) ? __ldg(g_row + base + c4) : 0.0f;
      }
    }
    float A = 0.f, D = 0.f;
    if (has_block) {
#pragma unroll
      for (int i = 0; i < EPL; ++i) {
        float tt;
        if (EPL * lig + i < n && classify(sort_key(x[i], mag), tt) == 1) {
          const float dr = M.drho(tt);
          const float chi = mag ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
          D += dr; A += dr * chi * g[i];
        }
      }
      A = group_sum<G, float>(A, mask);
      D = group_sum<G, float>(D, mask);
      if (mag) D += (float)(k - a0);
    }
    const float ratio = D > 0.0f ? A / D : 0.0f;
    // second pass: residuals about the fp32 mean (one fma each, no cancellation) restore what the
    // division rounded away; rho' can be 3/lambda, and an ulp of the mean times that shows
    float delta = 0.0f;
    if (has_block) {
      float A2 = 0.f;
#pragma unroll
      for (int i = 0; i < EPL; ++i) {
        float tt;
        if (EPL * lig + i < n && classify(sort_key(x[i], mag), tt) == 1) {
          const float chi = mag ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
          A2 += M.drho(tt) * fmaf(chi, g[i], -ratio);
        }
      }
      A2 = group_sum<G, float>(A2, mask);
      if (mag) A2 -= (float)(k - a0) * ratio;
      delta = D > 0.0f ? A2 / D : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
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
  float* o_row = P.out + row * (long long)n;
#pragma unroll
  for (int h = 0; h < EPL / 4; ++h) {
    const int base = EPL * lig + 4 * h;
    if (P.vec4) {
      if (base < n) reinterpret_cast<float4*>(o_row)[base >> 2] = make_float4(o[4 * h], o[4 * h + 1], o[4 * h + 2], o[4 * h + 3]);
    } else {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) if (base + c4 < n) o_row[base + c4] = o[4 * h + c4];
    }
  }
  if (flags && P.status) atomicOr(P.status, flags);
}

}  // namespace

// Forward pass or recomputing VJP for rows of 129..512 elements when no permutation is asked for.
cudaError_t launch_groupv(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  if (P.n > 256) {                           // one warp per row, 16 elements per lane
    P.N = 512;
    tk_groupv_kernel<32, 16><<<(unsigned)((P.rows + 3) / 4), 128, 0, stream>>>(P);
    return cudaGetLastError();
  }
  P.N = 256;                                 // 128 < n <= 256: one warp per row, 8 elements per lane
  tk_groupv_kernel<32, 8><<<(unsigned)((P.rows + 3) / 4), 128, 0, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace tk
