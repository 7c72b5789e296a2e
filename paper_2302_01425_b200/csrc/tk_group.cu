// tk_group.cu -- short rows (n <= 256): G lanes of a warp per row, 8 elements
// per lane, the row never leaves registers / a few hundred bytes of shared
// memory.  32/G rows per warp.
//
// Same steps as the block-per-row kernel (Prop. 5/6 reduction; Sec. 5):
//   packed (key, index) -> sorting network (19-comparator 8-sorter per lane,
//   bitonic merges across lanes by shuffles) -> exact single-block isotonic
//   solve (G-ary search on the monotone predicates, O(1) probes through prefix
//   sums staged in shared memory) -> dual map -> scatter through shared memory
//   -> coalesced store.  Used when the caller wants the permutation (perm_out, tk_argsort);
//   the default forward pass and every VJP sort the keys alone (tk_rows.cu).
#include "tk_common.cuh"
#include "tk_group_sort.cuh"

namespace tk {

namespace {

// 8 elements per lane: registers capped at 64 so that 8 blocks (32 warps) fit an SM and a 1024-block
// grid (16384 rows of 64) is a single wave on 148 SMs.
template <int G, int EPL>
__global__ void __launch_bounds__(128, EPL == 8 ? 8 : 3) tk_group_kernel(const Problem P) {
  constexpr int N = G * EPL;                  // padded row length
  constexpr int GROUPS = 128 / G;             // rows per thread block
  constexpr int STRIDE = N + N / EPL + 1;     // padded slots per array per row
  auto pad8 = [](int i) -> int { return pad_e<EPL>(i); };
  __shared__ float sm[GROUPS][4][STRIDE];     // [0] keys / staging, [1..3] prefix sums of d, d^2, d^3

  const int tid = threadIdx.x;
  const int grp = tid / G, lig = tid % G;
  const long long row = (long long)blockIdx.x * GROUPS + grp;
  if (row >= P.rows) return;                  // whole groups leave together
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << ((tid & 31) / G * G);
  const int n = P.n, k = P.k;
  const Math M = make_math_q24(P);
  const bool mag = M.mag;
  float* sk = sm[grp][0];
  float* p1 = sm[grp][1];
  float* p2 = sm[grp][2];
  float* p3 = sm[grp][3];

  const float* x_row = P.theta + row * (long long)n;
  unsigned long long r[EPL];
  bool bad = false;
  group_load_pack_e<EPL>(P, x_row, lig, mag, r, bad);

  group_sort_e<G, EPL>(r, lig, mask);         // lane `lig` now holds sorted ranks [EPL lig, EPL lig + EPL)

  if (P.perm_out) {
    int32_t* pr = P.perm_out + row * (long long)n;
#pragma unroll
    for (int i = 0; i < EPL; ++i) if (EPL * lig + i < n) pr[EPL * lig + i] = un_idx(r[i]);
  }
  if (P.sorted_out) {
    float* so = P.sorted_out + row * (long long)n;
#pragma unroll
    for (int i = 0; i < EPL; ++i) if (EPL * lig + i < n) so[EPL * lig + i] = un_key(r[i]);
  }
  int flags = bad ? TK_FLAG_NONFINITE : 0;
  if (P.what == W_ARGSORT) {
    if (flags && P.status) atomicOr(P.status, flags);
    return;
  }

#pragma unroll
  for (int i = 0; i < EPL; ++i) sk[pad8(EPL * lig + i)] = un_key(r[i]);
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
      const float di = un_key(r[i]) - piv;
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
        if (rk >= wl && rk < wh) { const float di = un_key(r[i]) - piv; o1 += di; const float d2 = di * di; o2 += d2; o3 += d2 * di; }
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
      if (rk >= a0 && rk < b0) { const float di = un_key(r[i]) - piv; f1 += di; const float d2 = di * di; f2 += d2; f3 += d2 * di; }
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

  const float wid = has_block ? M.width(piv + u) : 0.0f;
  auto y_of = [&](int rk, unsigned long long e) -> float {
    if (rk < a0) return mag ? M.vtop(un_key(e)) : 1.0f;
    if (rk < b0) return M.rho(fminf(fmaxf((un_key(e) - piv) - u, 0.0f), wid));
    return 0.0f;
  };
  __syncwarp(mask);      // all reads of sk[] done; it becomes the staging buffer
  float* stage = sk;
  float* o_row = P.out + row * (long long)n;

  {   // forward pass only: tk_vjp never asks for a permutation, so it never comes here
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      const int idx = un_idx(r[i]);
      if (EPL * lig + i < n && idx < n) {
        const float yv = y_of(EPL * lig + i, r[i]);
        stage[pad8(idx)] = (mag && un_neg(r[i])) ? -yv : yv;
      }
    }
    __syncwarp(mask);
#pragma unroll
    for (int h = 0; h < EPL / 4; ++h) {
      const int base = EPL * lig + 4 * h;
      if (P.vec4) {
        if (base < n) {
          float4 q = make_float4(stage[pad8(base)], stage[pad8(base + 1)], stage[pad8(base + 2)], stage[pad8(base + 3)]);
          if (P.mode == TK_TOPK) {
            float4 xx = __ldg(reinterpret_cast<const float4*>(x_row) + (base >> 2));
            q.x *= xx.x; q.y *= xx.y; q.z *= xx.z; q.w *= xx.w;
          }
          reinterpret_cast<float4*>(o_row)[base >> 2] = q;
        }
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          const int i = base + c4;
          if (i < n) { float q = stage[pad8(i)]; if (P.mode == TK_TOPK) q *= __ldg(x_row + i); o_row[i] = q; }
        }
      }
    }
  }
  if (flags && P.status) atomicOr(P.status, flags);
}

}  // namespace

cudaError_t launch_group(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  if (P.n > 256) {      // one warp per row, 16 elements per lane
    P.N = 512;
    const unsigned blocks = (unsigned)((P.rows + 3) / 4);
    tk_group_kernel<32, 16><<<blocks, 128, 0, stream>>>(P);
    return cudaGetLastError();
  }
  int G = 1;
  while (G * 8 < P.n) G <<= 1;
  P.N = G * 8;
  const long long groups = 128 / G;
  const unsigned blocks = (unsigned)((P.rows + groups - 1) / groups);
  switch (G) {
    case 1: tk_group_kernel<1, 8><<<blocks, 128, 0, stream>>>(P); break;
    case 2: tk_group_kernel<2, 8><<<blocks, 128, 0, stream>>>(P); break;
    case 4: tk_group_kernel<4, 8><<<blocks, 128, 0, stream>>>(P); break;
    case 8: tk_group_kernel<8, 8><<<blocks, 128, 0, stream>>>(P); break;
    case 16: tk_group_kernel<16, 8><<<blocks, 128, 0, stream>>>(P); break;
    default: tk_group_kernel<32, 8><<<blocks, 128, 0, stream>>>(P); break;
  }
  return cudaGetLastError();
}

}  // namespace tk
