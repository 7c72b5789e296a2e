// tk_rows.cu -- rows of up to 256 elements, the default forward pass and VJP.
//
// Every warp works alone on up to 32 rows (16 when n > 64, 8 when n > 128), in three phases:
//   1. in batches of 32/G rows (G lanes x 8 keys per row; one lane x 16 keys for 8 < n <= 16,
//      where the whole network then runs in registers): load, sort the 32-bit KEYS by the
//      shuffle network, leave the sorted row in the warp's shared memory;
//   2. lane r solves row r: the isotonic problem of Sec. 5 has at most one pooled block [a0, b0)
//      around ranks k-1 and k, and it is grown from that pair one rank at a time, pooling a
//      neighbour while it violates the order, on running power sums of d = key - pivot (see
//      solve_row_walk).  Up to 32 rows walk side by side, so the solve costs a warp a few
//      instructions per block member instead of a search replicated over the G lanes of every row;
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

template <int G, int E, int B, bool Q4, bool MAG>
__global__ void __launch_bounds__(kRowsThreads, E == 8 ? 6 : 4) tk_rows_kernel(const Problem P) {
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
  M.q4 = Q4; M.mag = MAG;
  int flags = 0;

  // the lane's E consecutive elements of a row (zeros past the row's end)
  auto load8 = [&](const float* base, bool live, float (&v)[E]) {
#pragma unroll
    for (int h = 0; h < E / 4; ++h) {
      const int e0 = E * lig + 4 * h;
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
  float xkeep[E];                                 // a single batch keeps its row for phase 3
#pragma unroll 1
  for (int b = 0; b < BATCHES; ++b) {
    const int rr = b * RPB + gw;
    const long long row = row0 + rr;
    const bool live = row < P.rows;
    float x[E], s[E];
    load8(P.theta + (live ? row : 0) * (long long)n, live, x);
    if (BATCHES == 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) xkeep[i] = x[i];
    }
    bool bad = false;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const bool in = E * lig + i < n;
      if (in && !isfinite(x[i])) bad = true;
      s[i] = in ? sort_key(x[i], MAG) : -INFINITY;       // slots past the row sort last
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
    float x[E];
    if (BATCHES == 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) x[i] = xkeep[i];
    } else {
      load8(P.theta + (live ? row : 0) * (long long)n, live, x);   // second read: L1 / L2
    }
    const float wid = has_block ? M.width(piv + u) : 0.0f;
    // class of a key: 2 capped (top singleton), 1 pooled, 0 zero; tt = key - gamma, clamped
    auto classify = [&](float key, float& tt) -> int {
      if (!has_block) { tt = 0.0f; return key >= c ? 2 : 0; }
      const float t = (key - piv) - u;
      tt = fminf(fmaxf(t, 0.0f), wid);
      return t >= wid ? 2 : (t > 0.0f ? 1 : 0);
    };
    float o[E];
    if (P.what == W_FWD) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
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
      float g[E];
      load8(P.gout + (live ? row : 0) * (long long)n, live, g);
      float A = 0.f, D = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        float tt;
        if (has_block && E * lig + i < n && classify(sort_key(x[i], MAG), tt) == 1) {
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
      for (int i = 0; i < E; ++i) {
        float tt;
        if (has_block && E * lig + i < n && classify(sort_key(x[i], MAG), tt) == 1) {
          const float chi = MAG ? (signbit(x[i]) ? -1.0f : 1.0f) : (P.mode == TK_TOPK ? x[i] : 1.0f);
          A2 += M.drho(tt) * fmaf(chi, g[i], -ratio);
        }
      }
      A2 = group_sum<G, float>(A2, mask);
      if (MAG && has_block) A2 -= (float)(k - a0) * ratio;
      const float delta = D > 0.0f ? A2 / D : 0.0f;
#pragma unroll
      for (int i = 0; i < E; ++i) {
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
    for (int h = 0; h < E / 4; ++h) {
      const int e0 = E * lig + 4 * h;
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

template <int G, int E, int B>
cudaError_t launch_rows_gb(const Problem& P, cudaStream_t stream) {
  const long long per_block = (long long)(kRowsThreads / 32) * RowsGeom<G, E, B>::R;
  const unsigned blocks = (unsigned)((P.rows + per_block - 1) / per_block);
  const bool mag = P.mode == TK_TOPKMAG;
  if (P.q4) {
    if (mag) tk_rows_kernel<G, E, B, true, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, E, B, true, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  } else {
    if (mag) tk_rows_kernel<G, E, B, false, true><<<blocks, kRowsThreads, 0, stream>>>(P);
    else tk_rows_kernel<G, E, B, false, false><<<blocks, kRowsThreads, 0, stream>>>(P);
  }
  return cudaGetLastError();
}

constexpr long long kWarpsToFill = 148 * 24;   // warps below which a launch leaves SMs short of work

// 8 keys per lane.  The most batches per warp that still leave kWarpsToFill warps, out of {1, 2, BMAX}.
template <int G, int BMAX>
cudaError_t launch_rows_g(const Problem& P, cudaStream_t stream) {
  constexpr int RPB = 32 / G;
  if (BMAX > 2 && P.rows / (RPB * BMAX) >= kWarpsToFill) return launch_rows_gb<G, 8, BMAX>(P, stream);
  if (BMAX >= 2 && P.rows / (RPB * 2) >= kWarpsToFill) return launch_rows_gb<G, 8, (BMAX >= 2 ? 2 : 1)>(P, stream);
  return launch_rows_gb<G, 8, 1>(P, stream);
}

}  // namespace

// Forward pass or recomputing VJP for rows of up to 256 elements when no permutation is asked for.
cudaError_t launch_rows(const Problem& P0, cudaStream_t stream) {
  Problem P = P0;
  if (P.n > 8 && P.n <= 16) {                  // one lane per row, 16 keys: the whole sort in registers
    P.N = 16;
    return launch_rows_gb<1, 16, 1>(P, stream);
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
