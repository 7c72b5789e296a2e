// tk_rows.cu -- rows of up to 256 elements, the default forward pass and VJP.
//
// Every warp works alone on up to 32 rows (16 when n > 64, 8 when n > 128), in three phases:
//   1. in batches of 32/G rows (G lanes x 8 elements per row): load, sort the 32-bit KEYS by the
//      shuffle network, leave the sorted row in the warp's shared memory;
//   2. lane r solves row r: the isotonic problem of Sec. 5 has at most one pooled block [a0, b0)
//      around ranks k-1 and k, and both edges are found by WALKING outwards from k with running
//      power sums of d = key - pivot (see solve_row_walk).  Up to 32 rows walk side by side, so
//      the solve costs a warp a few instructions per block member instead of a search replicated
//      over the G lanes of every row;
//   3. in the same batches: the results by value (given gamma and the cap width, the output and
//      the VJP of an element depend on its own key alone), stored where they were loaded.
// No index travels through the sort and nothing is scattered; the phases are separated by warp
// barriers only, so the other warps of the SM fill the latency of a warp that is walking.
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
// sk[i + i/8]).  F(tau) = #{capped at tau} - k + sum over the ranks strictly between the caps of
// rho(s_i - tau) / phi'(tau) is the monotone threshold function whose root is gamma.  Rank j > k
// joins the block while F(s_j) < 0; rank j < k-1 joins while F(vtop(s_j)) > 0.  Each edge is one
// flat loop: a step either moves the far end of the summed range (which only moves one way as j
// does) or tests j and moves on, so 32 lanes with different rows stay in one instruction stream.
template <bool Q4, bool MAG>
__device__ __forceinline__ void solve_row_walk(const float* sk, int n, int k, const Math& M, const Problem& P,
                                               RowSol& R) {
  auto key = [&](int i) -> float { return sk[i + (i >> 3)]; };
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
    const float W_hi = (piv == c) ? M.width(c) : c + M.width(c);
    const float W_lo = vtop_c - piv;
    const float il3 = P.inv_lam * P.inv_lam * P.inv_lam;
    float D1 = 0.f, D2 = 0.f, D3 = 0.f;
    auto add = [&](float d) { D1 += d; if (Q4) { const float d2 = d * d; D2 += d2; D3 = fmaf(d2, d, D3); } };
    auto sub = [&](float d) { D1 -= d; if (Q4) { const float d2 = d * d; D2 -= d2; D3 = fmaf(-d2, d, D3); } };
    // F at gamma = pivot + uu, ranks [r_hi, r_lo) between the caps with power sums E1..E3
    auto Fval = [&](float uu, int r_hi, int r_lo, float E1, float E2, float E3) -> float {
      const float cnt = (float)(r_lo - r_hi);
      float S;
      if (Q4) S = (((-cnt * uu + 3.0f * E1) * uu - 3.0f * E2) * uu + E3) * il3;
      else S = (E1 - cnt * uu) * P.inv_lam;
      if (MAG) S = S / (piv + uu);
      return (float)(r_hi - k) + S;
    };
    // ---- upper edge.  r_hi(j) = #{i < k : d_i >= d_j + width(s_j)} only grows with j: start it at
    // its least value (the window's upper end) and advance.
    {
      int r_hi = k;
      while (r_hi > 0) { const float d = key(r_hi - 1) - piv; if (d >= W_hi) break; add(d); --r_hi; }
      add(key(k) - piv);
      int j = k + 1;
      b0 = k + 1;
      float uu = 0.f, thr = 0.f;
      bool in_window = false;
      auto prep = [&]() {
        const float tau = key(min(j, n - 1));
        uu = tau - piv;
        in_window = (j < n) && (uu > W_lo) && !(MAG && !(tau > 0.0f));   // else at or below vtop(c)
        thr = uu + M.width(tau);
      };
      prep();
      while (in_window) {
        const float dr = key(min(r_hi, k - 1)) - piv;
        if (r_hi < k && dr >= thr) { sub(dr); ++r_hi; }
        else {
          if (!(Fval(uu, r_hi, j, D1, D2, D3) < 0.0f)) break;
          add(uu); ++j; b0 = j;
          prep();
        }
      }
    }
    // ---- lower edge.  r_lo(j) = k + #{i >= k : d_i > vtop(s_j) - pivot} only shrinks as j falls:
    // start it at its greatest value (the window's lower end) and retreat.
    a0 = k - 1;
    if (k >= 2) {
      D1 = 0.f; D2 = 0.f; D3 = 0.f;
      int r_lo = k;
      while (r_lo < n) { const float d = key(r_lo) - piv; if (!(d > W_lo)) break; add(d); ++r_lo; }
      add(key(k - 1) - piv);
      int j = k - 2;
      float dj = 0.f, uu = 0.f;
      bool open = false, valid = false;
      auto prep = [&]() {
        const float sj = key(max(j, 0));
        dj = sj - piv;
        open = (j >= 0) && !(dj >= W_hi);               // else capped whatever gamma is
        const float tau = M.vtop(sj);
        uu = tau - piv;
        valid = !(MAG && !(tau > 0.0f));
      };
      prep();
      while (open) {
        const float dl = key(max(r_lo - 1, k)) - piv;
        if (valid && r_lo > k && !(dl > uu)) { sub(dl); --r_lo; }
        else {
          if (valid) {
            const float dj2 = dj * dj;
            // F <= 0: rank j stays a top singleton, and so do all ranks above it
            if (Fval(uu, j, r_lo, D1 + dj, D2 + dj2, fmaf(dj2, dj, D3)) <= 0.0f) break;
          }
          a0 = j; add(dj); --j;
          prep();
        }
      }
    }
    // ---- block mean and central sums over [a0, b0), then the block value
    double s1 = 0.0;
    for (int i = a0; i < b0; ++i) s1 += (double)(key(i) - piv);
    const float cnt = (float)(b0 - a0), m = (float)(k - a0);
    const float mu = (float)(s1 / (double)cnt);
    float M2 = 0.f, M3 = 0.f;
    if (Q4) {
      for (int i = a0; i < b0; ++i) {
        const float e = (key(i) - piv) - mu;
        const float e2 = e * e;
        M2 += e2; M3 = fmaf(e2, e, M3);
      }
    }
    u = block_value<Q4, MAG>(P.lam, P.lam3, piv, cnt, m, mu, M2, M3);
    u = settle_offset(M, piv, u, a0, b0, n, key);
  }
  R.piv = piv; R.u = u; R.c = c; R.a0 = a0; R.b0 = b0; R.has_block = has_block ? 1 : 0;
}

constexpr int kRowsThreads = 128;

// B batches of 32/G rows per warp.  The most batches (32 rows per warp, 16 for n > 64, 8 for
// n > 128) cost the fewest instructions per row; fewer batches give a small problem enough warps
// to fill the machine.
template <int G, int B>
struct RowsGeom {
  static constexpr int N = 8 * G;                          // padded row length
  static constexpr int RPB = 32 / G;                       // rows per batch
  static constexpr int R = RPB * B;                        // rows per warp
  static constexpr int STRIDE = (N + G - 1) | 1;           // odd: lane r walking row r meets no bank conflict
};

template <int G, int B, bool Q4, bool MAG>
__global__ void __launch_bounds__(kRowsThreads, 6) tk_rows_kernel(const Problem P) {
  constexpr int RPB = RowsGeom<G, B>::RPB, R = RowsGeom<G, B>::R, BATCHES = B;
  constexpr int STRIDE = RowsGeom<G, B>::STRIDE;
  constexpr int WARPS = kRowsThreads / 32;
  __shared__ float sm[WARPS][R][STRIDE];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gw = lane / G, lig = lane % G;        // the lane's row within a batch, its place in the row
  constexpr unsigned kGroupBits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned mask = kGroupBits << (gw * G);
  const long long row0 = ((long long)blockIdx.x * WARPS + warp) * R;
  const int n = P.n, k = P.k;
  Math M = make_math(P);
  M.q4 = Q4; M.mag = MAG;
  int flags = 0;

  // the lane's 8 consecutive elements of a row (zeros past the row's end)
  auto load8 = [&](const float* base, bool live, float (&v)[8]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int e0 = 8 * lig + 4 * h;
      if (P.vec4) {
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live && e0 < n) q = __ldg(reinterpret_cast<const float4*>(base) + (e0 >> 2));
        v[4 * h] = q.x; v[4 * h + 1] = q.y; v[4 * h + 2] = q.z; v[4 * h + 3] = q.w;
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) v[4 * h + c4] = (live && e0 + c4 < n) ? __ldg(base + e0 + c4) : 0.0f;
      }
    }
  };

  // ---- phase 1: sort the keys of every row, batch by batch
#pragma unroll 1
  for (int b = 0; b < BATCHES; ++b) {
    const int rr = b * RPB + gw;
    const long long row = row0 + rr;
    const bool live = row < P.rows;
    float x[8], s[8];
    load8(P.theta + (live ? row : 0) * (long long)n, live, x);
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const bool in = 8 * lig + i < n;
      if (in && !isfinite(x[i])) bad = true;
      s[i] = in ? sort_key(x[i], MAG) : -INFINITY;       // slots past the row sort last
    }
    if (bad && live) flags |= TK_FLAG_NONFINITE;
    group_sort_keys<G, 8>(s, lig, mask);
    float* sk = sm[warp][rr];
#pragma unroll
    for (int i = 0; i < 8; ++i) sk[9 * lig + i] = s[i];   // rank 8 lig + i, one spare slot per 8
  }
  __syncwarp();

  // ---- phase 2: lane r solves row r
  RowSol mine;
  mine.piv = 0.f; mine.u = 0.f; mine.c = 0.f; mine.a0 = k; mine.b0 = k; mine.has_block = 0;
  if (lane < R && row0 + lane < P.rows) {
    solve_row_walk<Q4, MAG>(sm[warp][lane % R], n, k, M, P, mine);
    if (P.state_out) {
      tk_rowstate st;
      st.pivot = mine.has_block ? mine.piv : mine.c; st.offset = mine.u; st.a = mine.a0; st.b = mine.b0;
      P.state_out[row0 + lane] = st;
    }
  }
  __syncwarp();

  // ---- phase 3: results by value, in the original order
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
    float x[8];
    load8(P.theta + (live ? row : 0) * (long long)n, live, x);
    const float wid = has_block ? M.width(piv + u) : 0.0f;
    // class of a key: 2 capped (top singleton), 1 pooled, 0 zero; tt = key - gamma, clamped
    auto classify = [&](float key, float& tt) -> int {
      if (!has_block) { tt = 0.0f; return key >= c ? 2 : 0; }
      const float t = (key - piv) - u;
      tt = fminf(fmaxf(t, 0.0f), wid);
      return t >= wid ? 2 : (t > 0.0f ? 1 : 0);
    };
    float o[8];
    if (P.what == W_FWD) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float tt;
        const float key = sort_key(x[i], MAG);
        const int cls = classify(key, tt);
        float v = cls == 2 ? (MAG ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
        if (MAG) v = signbit(x[i]) ? -v : v;
        if (P.mode == TK_TOPK) v *= x[i];
        o[i] = v;
      }
    } else {
      // ---- VJP (Prop. 7): o_j = rho'_j (chi_j g_j - A/D) on the pooled block, by value
      float g[8];
      load8(P.gout + (live ? row : 0) * (long long)n, live, g);
      float A = 0.f, D = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float tt;
        if (has_block && 8 * lig + i < n && classify(sort_key(x[i], MAG), tt) == 1) {
          const float dr = M.drho(tt);
          const float chi = MAG ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
          D += dr; A += dr * chi * g[i];
        }
      }
      A = group_sum<G, float>(A, mask);
      D = group_sum<G, float>(D, mask);
      if (MAG && has_block) D += (float)(k - a0);
      const float ratio = D > 0.0f ? A / D : 0.0f;
      // second pass: residuals about the fp32 mean (one fma each, no cancellation) restore what
      // the division rounded away; rho' can be 3/lambda, and an ulp of the mean times that shows
      float A2 = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float tt;
        if (has_block && 8 * lig + i < n && classify(sort_key(x[i], MAG), tt) == 1) {
          const float chi = MAG ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
          A2 += M.drho(tt) * fmaf(chi, g[i], -ratio);
        }
      }
      A2 = group_sum<G, float>(A2, mask);
      if (MAG && has_block) A2 -= (float)(k - a0) * ratio;
      const float delta = D > 0.0f ? A2 / D : 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float tt;
        const float key = sort_key(x[i], MAG);
        const int cls = classify(key, tt);
        const float sgn = (MAG && signbit(x[i])) ? -1.0f : 1.0f;
        const float chi = MAG ? sgn : (P.mode == TK_TOPK ? x[i] : 1.0f);
        float v = 0.0f;
        if (cls == 1) v = M.drho(tt) * (fmaf(chi, g[i], -ratio) - delta);
        else if (cls == 2 && MAG) v = chi * g[i] * M.top_slope(key);
        v *= sgn;
        if (P.mode == TK_TOPK) v += g[i] * (cls == 2 ? 1.0f : (cls == 1 ? M.rho(tt) : 0.0f));
        o[i] = v;
      }
    }
    float* o_row = P.out + (live ? row : 0) * (long long)n;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int e0 = 8 * lig + 4 * h;
      if (P.vec4) {
        if (live && e0 < n) reinterpret_cast<float4*>(o_row)[e0 >> 2] = make_float4(o[4 * h], o[4 * h + 1], o[4 * h + 2], o[4 * h + 3]);
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) if (live && e0 + c4 < n) o_row[e0 + c4] = o[4 * h + c4];
      }
    }
  }
  if (flags && P.status) atomicOr(P.status, flags);
}

template <int G, int B>
cudaError_t launch_rows_gb(const Problem& P, cudaStream_t stream) {
  const long long per_block = (long long)(kRowsThreads / 32) * RowsGeom<G, B>::R;
  const unsigned blocks = (unsigned)((P.rows + per_block - 1) / per_block);
  const bool mag = P.mode == TK_TOPKMAG;
  if (P.q4) {
    if (mag) tk_rows_kernel<G, B, true, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, B, true, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  } else {
    if (mag) tk_rows_kernel<G, B, false, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, B, false, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  }
  return cudaGetLastError();
}

constexpr long long kWarpsToFill = 148 * 24;   // warps below which a launch leaves SMs short of work

// The most batches per warp that still leave kWarpsToFill warps, out of {1, 2, BMAX}.
template <int G, int BMAX>
cudaError_t launch_rows_g(const Problem& P, cudaStream_t stream) {
  constexpr int RPB = 32 / G;
  if (BMAX > 2 && P.rows / (RPB * BMAX) >= kWarpsToFill) return launch_rows_gb<G, BMAX>(P, stream);
  if (BMAX >= 2 && P.rows / (RPB * 2) >= kWarpsToFill) return launch_rows_gb<G, (BMAX >= 2 ? 2 : 1)>(P, stream);
  return launch_rows_gb<G, 1>(P, stream);
}

}  // namespace

// Forward pass or recomputing VJP for rows of up to 256 elements when no permutation is asked for.
cudaError_t launch_rows(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  int G = 1;
  while (G * 8 < P.n) G <<= 1;
  P.N = G * 8;
  switch (G) {
    case 1: return launch_rows_g<1, 1>(P, stream);
    case 2: return launch_rows_g<2, 2>(P, stream);
    case 4: return launch_rows_g<4, 4>(P, stream);
    case 8: return launch_rows_g<8, 8>(P, stream);
    case 16: return launch_rows_g<16, 8>(P, stream);
    default: return launch_rows_g<32, 8>(P, stream);
  }
}

}  // namespace tk
