// tk_vjp_state.cu -- VJP from the row state saved by the forward pass: rows too long for registers.
//
// Prop. 7 makes the Jacobian of the isotonic solution block diagonal with one
// rank-one block per pooled block; with w = 1_k there is at most one pooled
// block per row, and its members are exactly the keys strictly between gamma
// and gamma + width (width: the key distance at which rho reaches phi'(gamma)).
// Membership is therefore decided from the key alone and no permutation is
// needed: two row reductions (A = sum rho' chi g, D = sum rho') and one
// elementwise pass.  Traffic: theta and g in, grad out (12 B per element).
#include "tk_common.cuh"

namespace tk {

// rows held in registers (tk_vjp_team.cu)
int vjp_team_max_n();
cudaError_t launch_vjp_team(const Problem& P, cudaStream_t stream);

namespace {

// JVP (P.jvp): J is symmetric for the mask and the magnitude modes (in sorted coordinates it is
// diag(rho') - rho' rho'^T / D, and signs enter as S J S), so the same code serves.  For topk,
// y = theta o mask(theta): the VJP is g o mask + J_mask^T (theta o g), the JVP is v o mask +
// theta o (J_mask v): the weight theta moves from inside the block mean to outside it.
struct RowCtx {
  float pivot, offset, wid;
  bool has_block;
  int m;            // members of the pooled block with w = 1 (ranks a..k-1)
};

__device__ __forceinline__ RowCtx load_ctx(const Problem& P, const Math& M, long long row) {
  tk_rowstate st = P.state_in[row];
  RowCtx c;
  c.pivot = st.pivot; c.offset = st.offset;
  c.has_block = st.b > st.a;
  c.wid = c.has_block ? M.width(st.pivot + st.offset) : 0.0f;
  c.m = P.k - st.a;
  return c;
}

// class of an element: 0 bottom singleton, 1 pooled, 2 top singleton; tt = key - gamma clamped
__device__ __forceinline__ int classify(const RowCtx& c, float key, float& tt) {
  float d = key - c.pivot;
  if (!c.has_block) { tt = 0.0f; return d >= 0.0f ? 2 : 0; }
  float t = d - c.offset;
  tt = fminf(fmaxf(t, 0.0f), c.wid);
  if (t >= c.wid) return 2;
  return t > 0.0f ? 1 : 0;
}

// The mean A/D is needed to a relative accuracy of its DISTANCE from chi g, not of itself: rho' can
// be 3/lambda, and one ulp of A/D times that is above 1e-5.  Two ways to get it:
//  * rows held in registers: a second pass over the registers sums the residuals rho' (chi g - r0)
//    about the fp32 mean r0 of the first pass; each residual is one fma (no cancellation), and
//    the correction delta = (sum - m r0)/D restores what the division rounded away;
//  * rows streamed from memory: A and D are accumulated in fp64 (products of floats are exact
//    there), the mean is split into r0 = fl(mean) and delta = mean - r0.
// Either way the result is rho' ((chi g - r0) - delta).
__device__ __forceinline__ void accumulate_f64(const Problem& P, const Math& M, const RowCtx& c, float x,
                                               float g, double& A, double& D) {
  float tt;
  float key = sort_key(x, M.mag);
  if (classify(c, key, tt) == 1) {
    double dr = (double)M.drho(tt);
    float chi = M.mag ? (signbit(x) ? -1.0f : 1.0f) : ((P.mode == TK_TOPK && !P.jvp) ? x : 1.0f);
    D += dr;
    A += dr * ((double)chi * (double)g);
  }
}

__device__ __forceinline__ float finish(const Problem& P, const Math& M, const RowCtx& c, float x,
                                        float g, float ratio, float delta) {
  float tt;
  float key = sort_key(x, M.mag);
  int cls = classify(c, key, tt);
  float sgn = (M.mag && signbit(x)) ? -1.0f : 1.0f;
  const bool jt = P.mode == TK_TOPK && P.jvp;
  float chi = M.mag ? sgn : ((P.mode == TK_TOPK && !jt) ? x : 1.0f);
  float o = 0.0f;
  if (cls == 1) o = (jt ? x : 1.0f) * M.drho(tt) * (fmaf(chi, g, -ratio) - delta);
  else if (cls == 2 && M.mag) o = chi * g * M.top_slope(key);
  o *= sgn;
  if (P.mode == TK_TOPK) {
    float y = cls == 2 ? 1.0f : (cls == 1 ? M.rho(tt) : 0.0f);
    o += g * y;
  }
  return o;
}

// one thread block per row
template <bool GEN>
__global__ void __launch_bounds__(256) tk_vjp_state_cta(const Problem P) {
  __shared__ double red[2][8];
  Math M = make_math(P);
  M.gen = GEN;
  const int t = threadIdx.x, T = blockDim.x, lane = t & 31, warp = t >> 5;
  const long long row = blockIdx.x;
  const int n = P.n;
  const RowCtx c = load_ctx(P, M, row);
  const float* x_row = P.theta + row * (long long)n;
  const float* g_row = P.gout + row * (long long)n;
  float* o_row = P.out + row * (long long)n;
  double A = 0.0, D = 0.0;
  if (c.has_block) {           // uniform per row
    if (P.vec4) {
      const float4* x4 = reinterpret_cast<const float4*>(x_row);
      const float4* g4 = reinterpret_cast<const float4*>(g_row);
      for (int v = t; 4 * v < n; v += T) {
        float4 x = __ldg(x4 + v), g = __ldg(g4 + v);
        accumulate_f64(P, M, c, x.x, g.x, A, D); accumulate_f64(P, M, c, x.y, g.y, A, D);
        accumulate_f64(P, M, c, x.z, g.z, A, D); accumulate_f64(P, M, c, x.w, g.w, A, D);
      }
    } else {
      for (int i = t; i < n; i += T) accumulate_f64(P, M, c, __ldg(x_row + i), __ldg(g_row + i), A, D);
    }
    A = warp_sum(A); D = warp_sum(D);
    if (lane == 0) { red[0][warp] = A; red[1][warp] = D; }
    __syncthreads();
    A = 0.0; D = 0.0;
    for (int w = 0; w < (T >> 5); ++w) { A += red[0][w]; D += red[1][w]; }
    if (M.mag) D += (double)c.m;
  }
  const double mean = D > 0.0 ? A / D : 0.0;
  const float ratio = (float)mean, delta = (float)(mean - (double)ratio);
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
    const float4* g4 = reinterpret_cast<const float4*>(g_row);
    float4* o4 = reinterpret_cast<float4*>(o_row);
    for (int v = t; 4 * v < n; v += T) {
      float4 x = __ldg(x4 + v), g = __ldg(g4 + v), o;
      o.x = finish(P, M, c, x.x, g.x, ratio, delta); o.y = finish(P, M, c, x.y, g.y, ratio, delta);
      o.z = finish(P, M, c, x.z, g.z, ratio, delta); o.w = finish(P, M, c, x.w, g.w, ratio, delta);
      o4[v] = o;
    }
  } else {
    for (int i = t; i < n; i += T) o_row[i] = finish(P, M, c, __ldg(x_row + i), __ldg(g_row + i), ratio, delta);
  }
}

// Rows held in global memory: per-tile partial sums, then every block re-reduces them
// (no atomics, so results do not depend on scheduling) and finishes its own tile.
__global__ void __launch_bounds__(256) tk_vjp_long_partial(const Problem P, double2* partial, int tiles) {
  __shared__ double red[2][8];
  const Math M = make_math_q24(P);
  const long long row = blockIdx.y;
  const int tile = blockIdx.x, t = threadIdx.x, n = P.n;
  const RowCtx c = load_ctx(P, M, row);
  double A = 0.0, D = 0.0;
  if (c.has_block) {
    const float* x_row = P.theta + row * (long long)n;
    const float* g_row = P.gout + row * (long long)n;
    const int start = tile * kLongTile;
    if (P.vec4) {                               // n % 4 == 0 and aligned rows: 128-bit loads
      const float4* x4 = reinterpret_cast<const float4*>(x_row + start);
      const float4* g4 = reinterpret_cast<const float4*>(g_row + start);
#pragma unroll
      for (int j = 0; j < kLongTile / 1024; ++j) {
        const int v = j * 256 + t;
        if (start + 4 * v < n) {
          const float4 x = __ldg(x4 + v), g = __ldg(g4 + v);
          accumulate_f64(P, M, c, x.x, g.x, A, D); accumulate_f64(P, M, c, x.y, g.y, A, D);
          accumulate_f64(P, M, c, x.z, g.z, A, D); accumulate_f64(P, M, c, x.w, g.w, A, D);
        }
      }
    } else {
#pragma unroll 4
      for (int j = 0; j < kLongTile / 256; ++j) {
        const int i = start + j * 256 + t;
        if (i < n) accumulate_f64(P, M, c, __ldg(x_row + i), __ldg(g_row + i), A, D);
      }
    }
  }
  A = warp_sum(A); D = warp_sum(D);
  if ((t & 31) == 0) { red[0][t >> 5] = A; red[1][t >> 5] = D; }
  __syncthreads();
  if (t == 0) {
    double a = 0.0, d = 0.0;
    for (int w = 0; w < 8; ++w) { a += red[0][w]; d += red[1][w]; }
    partial[row * (long long)tiles + tile] = make_double2(a, d);
  }
}

__global__ void __launch_bounds__(256) tk_vjp_long_finish(const Problem P, const double2* partial, int tiles) {
  __shared__ double red[2][8];
  const Math M = make_math_q24(P);
  const long long row = blockIdx.y;
  const int tile = blockIdx.x, t = threadIdx.x, n = P.n;
  const RowCtx c = load_ctx(P, M, row);
  double A = 0.0, D = 0.0;
  for (int i = t; i < tiles; i += 256) { double2 v = partial[row * (long long)tiles + i]; A += v.x; D += v.y; }
  A = warp_sum(A); D = warp_sum(D);
  if ((t & 31) == 0) { red[0][t >> 5] = A; red[1][t >> 5] = D; }
  __syncthreads();
  A = 0.0; D = 0.0;
  for (int w = 0; w < 8; ++w) { A += red[0][w]; D += red[1][w]; }
  if (M.mag && c.has_block) D += (double)c.m;
  const double mean = D > 0.0 ? A / D : 0.0;
  const float ratio = (float)mean, delta = (float)(mean - (double)ratio);
  const float* x_row = P.theta + row * (long long)n;
  const float* g_row = P.gout + row * (long long)n;
  float* o_row = P.out + row * (long long)n;
  const int start = tile * kLongTile;
  if (P.vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row + start);
    const float4* g4 = reinterpret_cast<const float4*>(g_row + start);
    float4* o4 = reinterpret_cast<float4*>(o_row + start);
#pragma unroll
    for (int j = 0; j < kLongTile / 1024; ++j) {
      const int v = j * 256 + t;
      if (start + 4 * v < n) {
        const float4 x = __ldg(x4 + v), g = __ldg(g4 + v);
        float4 o;
        o.x = finish(P, M, c, x.x, g.x, ratio, delta); o.y = finish(P, M, c, x.y, g.y, ratio, delta);
        o.z = finish(P, M, c, x.z, g.z, ratio, delta); o.w = finish(P, M, c, x.w, g.w, ratio, delta);
        o4[v] = o;
      }
    }
    return;
  }
#pragma unroll 4
  for (int j = 0; j < kLongTile / 256; ++j) {
    const int i = start + j * 256 + t;
    if (i < n) o_row[i] = finish(P, M, c, __ldg(x_row + i), __ldg(g_row + i), ratio, delta);
  }
}

}  // namespace

// scratch: rows * ceil(n / kLongTile) * 16 bytes
cudaError_t launch_vjp_state_long(const Problem& P, void* scratch, cudaStream_t stream) {
  const int tiles = (P.n + kLongTile - 1) / kLongTile;
  const dim3 grid((unsigned)tiles, (unsigned)P.rows);
  double2* partial = static_cast<double2*>(scratch);
  tk_vjp_long_partial<<<grid, 256, 0, stream>>>(P, partial, tiles);
  tk_vjp_long_finish<<<grid, 256, 0, stream>>>(P, partial, tiles);
  return cudaGetLastError();
}

cudaError_t launch_vjp_state(const Problem& P, cudaStream_t stream) {
  // rows of up to 16384 elements are held in registers (tk_vjp_team.cu); longer ones are streamed twice
  if (P.n <= vjp_team_max_n()) return launch_vjp_team(P, stream);
  const bool gen = P.qm1 > 0.0f;
  (gen ? tk_vjp_state_cta<true> : tk_vjp_state_cta<false>)<<<(unsigned)P.rows, 256, 0, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace tk
