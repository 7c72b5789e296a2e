// tk_vjp_team.cu -- VJP / JVP from the row state saved by the forward pass, rows of up to 32768
// elements held in registers (above 16384 in the registers of a cluster of four thread blocks).
//
// Prop. 7 makes the Jacobian of the isotonic solution block diagonal with one rank-one block per
// pooled block; with w = 1_k there is at most one pooled block per row, and its members are
// exactly the keys strictly between gamma and gamma + width (width: the key distance at which rho
// reaches phi'(gamma)).  Membership is decided from the key alone, so no permutation is needed:
//   o_j = rho'_j (chi_j g_j - A / D),  A = sum_B rho' chi g,  D = sum_B rho' (+ m for phi even),
// two sums over the row and one elementwise pass.  Traffic: theta and g in, grad out (12 B per
// element); theta and g are read once, into registers.
//
// A row is held by a team of T lanes (G lanes of a warp, or W warps), E elements per lane: chunk c
// of team lane tl is float4 number c * T + tl of the row (T * 16 contiguous bytes per row and
// instruction).  Mode and q are template parameters: the mask kernels carry nothing of the
// magnitude mode's cube roots.
//
// The mean A / D is needed to a relative accuracy of its DISTANCE from chi g, not of itself: rho'
// can be 3 / lambda, and one ulp of A / D times that is above 1e-5.  A second pass over the
// registers sums the residuals rho' (chi g - r0) about the fp32 mean r0 of the first pass (one
// fma each, no cancellation); delta = (sum - m r0) / D restores what the division rounded away,
// and the result is rho' ((chi g - r0) - delta).
//
// JVP (P.jvp): J is symmetric for the mask and the magnitude modes (in sorted coordinates it is
// diag(rho') - rho' rho'^T / D, and signs enter as S J S), so the same code serves.  For topk,
// y = theta o mask(theta): the VJP is g o mask + J_mask^T (theta o g), the JVP is v o mask +
// theta o (J_mask v): the weight theta moves from inside the block mean to outside it.
#include <cooperative_groups.h>

#include "tk_team.cuh"

namespace cg = cooperative_groups;

namespace tk {

namespace {

// warps per SM the register budget is set for: the mask keeps two arrays beside theta and g, the other modes three
constexpr int vt_min_blocks(int E, int W, int MODE) {
  return team_min_blocks(E >= 32 ? 16 : (MODE == TK_MASK ? 32 : 24), W);
}

// The sums of a row shared by the CL thread blocks of a cluster: each block leaves its own total in its
// shared memory, a cluster barrier, then every block adds the CL totals in rank order (same order, same
// result in every block).
template <int NV, int CL>
__device__ __forceinline__ void vt_cluster_sum(float (&v)[NV], float* slot, cg::cluster_group& cluster) {
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) slot[i] = v[i];
  }
  cluster.sync();
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = 0.0f;
#pragma unroll
  for (int r = 0; r < CL; ++r) {
    const float* peer = cluster.map_shared_rank(slot, (unsigned)r);
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] += peer[i];
  }
}

// QM: 0 = q is 2, 1 = q is 4, 2 = any other q (rho' through powf).  MODE: tk_mode.  CL: thread blocks
// per row (above 1: a cluster of CL blocks, each with its share of the row in its registers).
template <int G, int E, int W, int QM, int MODE, int CL>
__global__ void __launch_bounds__(team_threads(W), vt_min_blocks(E, W, MODE)) tk_vjp_team_kernel(const Problem P) {
  extern __shared__ float vt_smem[];
  static_assert(W == 1 || G == 32, "several warps per row: every lane of them belongs to the row");
  static_assert(CL == 1 || W >= kTeamWarps, "a cluster shares one row: one team per block");
  constexpr int BW = kTeamWarps > W ? kTeamWarps : W;
  constexpr int TEAMS = BW / W;
  constexpr int R = W > 1 ? 1 : 32 / G;
  constexpr int T = G * W * CL;
  constexpr int CH = E / 4;
  constexpr bool MAG = MODE == TK_TOPKMAG, TOPK = MODE == TK_TOPK;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int team = warp / W, wit = warp % W;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned crank = CL > 1 ? cluster.block_rank() : 0u;
  const long long row0 = ((long long)(blockIdx.x / CL) * TEAMS + team) * R;
  if (row0 >= P.rows) return;                  // the whole team (CL > 1: the grid has exactly CL blocks per row)
  const int n = P.n;
  const int rl = lane / G, lig = lane % G;
  const long long row = row0 + rl;
  const bool row_ok = row < P.rows;
  const long long row_c = row_ok ? row : P.rows - 1;    // a group past the last row repeats it, stores nothing
  const int tl = (W > 1 ? wit * 32 + lane : lig) + (CL > 1 ? (int)crank * (W * 32) : 0);
  float* red = vt_smem + team * (2 * W * 4);
  const int bar = 1 + team;
  Math M = make_math(P);
  M.q4 = QM == 1; M.gen = QM == 2; M.mag = MAG;          // compile-time constants from here on
  const float* x_row = P.theta + row_c * (long long)n;
  const float* g_row = P.gout + row_c * (long long)n;
  float* o_row = P.out + row_c * (long long)n;

  // ---- theta and g: every load is unconditional (a chunk past the row re-reads its start)
  float x[E], g[E];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int p0 = 4 * (c * T + tl);
    if (P.vec4) {
      const int pc = p0 < n ? p0 : 0;
      float4 xv = make_float4(0.f, 0.f, 0.f, 0.f), gv = xv;
      if (TK_IN_BOUNDS(row_c * (long long)n + pc, 4, P.rows * (long long)n, P.status)) {
        xv = __ldg(reinterpret_cast<const float4*>(x_row + pc));
        gv = __ldg(reinterpret_cast<const float4*>(g_row + pc));
      }
      x[4 * c] = xv.x; x[4 * c + 1] = xv.y; x[4 * c + 2] = xv.z; x[4 * c + 3] = xv.w;
      g[4 * c] = gv.x; g[4 * c + 1] = gv.y; g[4 * c + 2] = gv.z; g[4 * c + 3] = gv.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pc = p0 + j < n ? p0 + j : 0;
        const bool okb = TK_IN_BOUNDS(row_c * (long long)n + pc, 1, P.rows * (long long)n, P.status);
        x[4 * c + j] = okb ? __ldg(x_row + pc) : 0.0f;
        g[4 * c + j] = okb ? __ldg(g_row + pc) : 0.0f;
      }
    }
  }
  tk_rowstate st;
  st.pivot = 0.0f; st.offset = 0.0f; st.a = P.k; st.b = P.k;
  if (TK_IN_BOUNDS(row_c, 1, P.rows, P.status)) st = P.state_in[row_c];
  const bool has_block = st.b > st.a;
  const float piv = st.pivot, off = st.offset;
  const float wid = has_block ? M.width(piv + off) : 0.0f;
  const float fm = (float)(P.k - st.a);        // members of the pooled block with w = 1
  const bool jt = TOPK && P.jvp;               // topk JVP: theta multiplies outside the block mean

  // ---- one classification per element: w = sign * rho' on the pooled block (else 0) and the part of
  // the result that does not depend on the block mean
  float w[E], fixed[E];
  float AD[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const int idx = 4 * ((i >> 2) * T + tl) + (i & 3);
    const float xv = x[i], gv = g[i];
    const float key = MAG ? fabsf(xv) : xv;
    const float d = key - piv;
    const float t = d - off;
    const bool in = idx < n;
    const bool top = in && (has_block ? t >= wid : d >= 0.0f);
    const bool mid = in && has_block && t > 0.0f && !top;
    const float tt = fminf(fmaxf(t, 0.0f), wid);
    const float sgn = (MAG && signbit(xv)) ? -1.0f : 1.0f;
    const float chi = MAG ? sgn : ((TOPK && !jt) ? xv : 1.0f);
    const float dr = mid ? M.drho(tt) : 0.0f;
    float f = 0.0f;
    if (MAG) f = top ? gv * M.top_slope(key) : 0.0f;          // sgn chi = 1 there
    if (TOPK) f = gv * (top ? 1.0f : (mid ? M.rho(tt) : 0.0f));
    w[i] = sgn * dr;
    fixed[i] = f;
    AD[0] = fmaf(dr * chi, gv, AD[0]);
    AD[1] += dr;
  }
  float ratio = 0.0f, delta = 0.0f;
  if (__any_sync(0xffffffffu, has_block)) {    // the warps of a row agree: same row state
    uint32_t none = 0;
    team_allsum<G, W, 2>(AD, none, red, wit, lane, bar);
    float* xch = vt_smem + TEAMS * (2 * W * 4);              // CL == 2: two slots of four words
    if (CL > 1) vt_cluster_sum<2, CL>(AD, xch, cluster);
    float D = AD[1];
    if (MAG) D += fm;
    const bool ok = has_block && D > 0.0f;
    ratio = ok ? AD[0] / D : 0.0f;
    float A2[1] = {0.f};
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float xv = x[i];
      const float sgn = (MAG && signbit(xv)) ? -1.0f : 1.0f;
      const float chi = MAG ? sgn : ((TOPK && !jt) ? xv : 1.0f);
      A2[0] = fmaf(fabsf(w[i]), fmaf(chi, g[i], -ratio), A2[0]);   // |w| = rho'
    }
    team_allsum<G, W, 1>(A2, none, red + W * 4, wit, lane, bar);
    if (CL > 1) {
      vt_cluster_sum<1, CL>(A2, xch + 4, cluster);
      cluster.sync();                          // no block leaves while the other may still read its slot
    }
    if (MAG) A2[0] -= fm * ratio;
    delta = ok ? A2[0] / D : 0.0f;
  }
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int p0 = 4 * (c * T + tl);
    float o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = 4 * c + j;
      const float xv = x[i];
      const float sgn = (MAG && signbit(xv)) ? -1.0f : 1.0f;
      const float chi = MAG ? sgn : ((TOPK && !jt) ? xv : 1.0f);
      o[j] = fmaf(w[i] * (jt ? xv : 1.0f), fmaf(chi, g[i], -ratio) - delta, fixed[i]);
    }
    if (P.vec4) {
      if (row_ok && p0 < n && TK_IN_BOUNDS(row_c * (long long)n + p0, 4, P.rows * (long long)n, P.status))
        *reinterpret_cast<float4*>(o_row + p0) = make_float4(o[0], o[1], o[2], o[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (row_ok && p0 + j < n && TK_IN_BOUNDS(row_c * (long long)n + p0 + j, 1, P.rows * (long long)n, P.status)) o_row[p0 + j] = o[j];
    }
  }
}

template <int G, int E, int W, int QM, int MODE, int CL>
cudaError_t vt_launch(const Problem& P, cudaStream_t stream) {
  constexpr int BW = kTeamWarps > W ? kTeamWarps : W;
  constexpr int TEAMS = BW / W;
  constexpr int smem = (TEAMS * 2 * W * 4 + (CL > 1 ? 8 : 0)) * (int)sizeof(float);
  constexpr long long rows_per_block = (long long)TEAMS * (W > 1 ? 1 : 32 / G);
  if (CL == 1) {
    const unsigned blocks = (unsigned)((P.rows + rows_per_block - 1) / rows_per_block);
    tk_vjp_team_kernel<G, E, W, QM, MODE, CL><<<blocks, BW * 32, smem, stream>>>(P);
    return cudaGetLastError();
  }
  // CL thread blocks per row, launched as a cluster
  if (P.rows > 0x3fffffffLL) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(P.rows * CL));
  cfg.blockDim = dim3(BW * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tk_vjp_team_kernel<G, E, W, QM, MODE, CL>, P);
}

template <int G, int E, int W, int CL = 1>
cudaError_t vt_launch_mode(const Problem& P, cudaStream_t stream) {
  const int qm = P.qm1 > 0.0f ? 2 : (P.q4 ? 1 : 0);
  switch (P.mode) {
    case TK_MASK:
      return qm == 0 ? vt_launch<G, E, W, 0, TK_MASK, CL>(P, stream)
                     : (qm == 1 ? vt_launch<G, E, W, 1, TK_MASK, CL>(P, stream) : vt_launch<G, E, W, 2, TK_MASK, CL>(P, stream));
    case TK_TOPK:
      return qm == 0 ? vt_launch<G, E, W, 0, TK_TOPK, CL>(P, stream)
                     : (qm == 1 ? vt_launch<G, E, W, 1, TK_TOPK, CL>(P, stream) : vt_launch<G, E, W, 2, TK_TOPK, CL>(P, stream));
    default:
      return qm == 0 ? vt_launch<G, E, W, 0, TK_TOPKMAG, CL>(P, stream)
                     : (qm == 1 ? vt_launch<G, E, W, 1, TK_TOPKMAG, CL>(P, stream) : vt_launch<G, E, W, 2, TK_TOPKMAG, CL>(P, stream));
  }
}

}  // namespace

int vjp_team_max_n() { return 32768; }

// VJP (or JVP) from saved row state for rows of up to vjp_team_max_n() elements.
cudaError_t launch_vjp_team(const Problem& P, cudaStream_t stream) {
  const int n = P.n;
  if (n <= 8) return vt_launch_mode<1, 8, 1>(P, stream);
  if (n <= 16) return vt_launch_mode<1, 16, 1>(P, stream);
  if (n <= 32) return vt_launch_mode<2, 16, 1>(P, stream);
  if (n <= 64) return vt_launch_mode<4, 16, 1>(P, stream);
  if (n <= 128) return vt_launch_mode<8, 16, 1>(P, stream);
  if (n <= 256) return vt_launch_mode<16, 16, 1>(P, stream);
  if (n <= 512) return vt_launch_mode<32, 16, 1>(P, stream);
  if (n <= 1024) return vt_launch_mode<32, 8, 4>(P, stream);
  if (n <= 2048) return vt_launch_mode<32, 16, 4>(P, stream);
  if (n <= 4096) return vt_launch_mode<32, 16, 8>(P, stream);
  if (n <= 8192) return vt_launch_mode<32, 16, 16>(P, stream);
  if (n <= 16384) return vt_launch_mode<32, 32, 16>(P, stream);
  return vt_launch_mode<32, 16, 16, 4>(P, stream);     // a cluster of four thread blocks per row (two were slower: one block per SM; eight too)
}

}  // namespace tk
