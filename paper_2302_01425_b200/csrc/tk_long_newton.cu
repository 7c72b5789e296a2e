// tk_long_newton.cu -- the sort-free forward pass for a few very long rows (the magnitude-pruning
// row: one row of millions of weights).
//
// The same iteration as tk_newton.cu (tk_newton_core.cuh: Newton on the pieces of the threshold
// function, whose root is the value of the single pooled block of Sec. 5), with the row in global
// memory instead of registers: every pass streams the row once -- from L2 after the first pass,
// a 16 MB row fits it several times over -- each thread block reduces its share of the counts and
// power sums, the blocks meet at a grid barrier (cooperative launch: all blocks are resident),
// and every block then adds the per-block partial sums in the same order and takes the same
// step.  Two partial-sum buffers alternate, so one grid barrier per pass is enough.  No sort, no
// histogram: 5 to 10 passes of 2 to 3 microseconds instead of four radix passes over (key, index)
// pairs.
#include <cooperative_groups.h>

#include "tk_newton_core.cuh"

namespace cg = cooperative_groups;

namespace tk {

namespace {

constexpr int kLnThreads = 256;
constexpr int kLnSlots = 8;                 // words per block and buffer: three sums and two counts (5 used)

struct LnAcc {
  float v0, v1, v2;
  uint32_t cnt, cnt2;
};

// Sum over the whole grid: block tree, one slot per block in `buf`, grid barrier, then every block adds
// all slots in the same order (thread t takes slots t, t + 256, ...; then the same block tree).
__device__ __forceinline__ LnAcc ln_grid_sum(LnAcc a, float* buf, float* sh, cg::grid_group& grid) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  auto block_sum = [&](LnAcc x) -> LnAcc {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      x.v0 += __shfl_xor_sync(0xffffffffu, x.v0, o);
      x.v1 += __shfl_xor_sync(0xffffffffu, x.v1, o);
      x.v2 += __shfl_xor_sync(0xffffffffu, x.v2, o);
      x.cnt += __shfl_xor_sync(0xffffffffu, x.cnt, o);
      x.cnt2 += __shfl_xor_sync(0xffffffffu, x.cnt2, o);
    }
    __syncthreads();                           // sh may still be read from the sum before
    if (lane == 0) {
      sh[warp * 5] = x.v0; sh[warp * 5 + 1] = x.v1; sh[warp * 5 + 2] = x.v2;
      sh[warp * 5 + 3] = __uint_as_float(x.cnt); sh[warp * 5 + 4] = __uint_as_float(x.cnt2);
    }
    __syncthreads();
    LnAcc r{0.f, 0.f, 0.f, 0u, 0u};
#pragma unroll
    for (int w = 0; w < kLnThreads / 32; ++w) {
      r.v0 += sh[w * 5]; r.v1 += sh[w * 5 + 1]; r.v2 += sh[w * 5 + 2];
      r.cnt += __float_as_uint(sh[w * 5 + 3]); r.cnt2 += __float_as_uint(sh[w * 5 + 4]);
    }
    return r;
  };
  const LnAcc b = block_sum(a);
  if (t == 0) {
    float* s = buf + (size_t)blockIdx.x * kLnSlots;
    s[0] = b.v0; s[1] = b.v1; s[2] = b.v2; s[3] = __uint_as_float(b.cnt); s[4] = __uint_as_float(b.cnt2);
  }
  grid.sync();
  LnAcc p{0.f, 0.f, 0.f, 0u, 0u};
  for (int i = t; i < (int)gridDim.x; i += kLnThreads) {
    const float* s = buf + (size_t)i * kLnSlots;
    p.v0 += __ldcg(s); p.v1 += __ldcg(s + 1); p.v2 += __ldcg(s + 2);
    p.cnt += __float_as_uint(__ldcg(s + 3)); p.cnt2 += __float_as_uint(__ldcg(s + 4));
  }
  return block_sum(p);
}

// smallest value over the grid (same scheme; buf slot 0)
__device__ __forceinline__ float ln_grid_min(float a, float* buf, float* sh, cg::grid_group& grid) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  auto block_min = [&](float x) -> float {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fminf(x, __shfl_xor_sync(0xffffffffu, x, o));
    __syncthreads();
    if (lane == 0) sh[warp] = x;
    __syncthreads();
    float r = sh[0];
#pragma unroll
    for (int w = 1; w < kLnThreads / 32; ++w) r = fminf(r, sh[w]);
    return r;
  };
  const float b = block_min(a);
  if (t == 0) buf[(size_t)blockIdx.x * kLnSlots] = b;
  grid.sync();
  float p = INFINITY;
  for (int i = t; i < (int)gridDim.x; i += kLnThreads) p = fminf(p, __ldcg(buf + (size_t)i * kLnSlots));
  return block_min(p);
}

// f(key, index) over this thread's share of the row: float4 chunks, grid-strided
template <bool MAG, class F>
__device__ __forceinline__ void ln_for_each(const float* x_row, int n, int vec4, int32_t* status, F f) {
  const long long stride = (long long)gridDim.x * kLnThreads;
  const long long first = (long long)blockIdx.x * kLnThreads + threadIdx.x;
  if (vec4) {
    const float4* x4 = reinterpret_cast<const float4*>(x_row);
    for (long long v = first; 4 * v < n; v += stride) {
      if (!TK_IN_BOUNDS(4 * v, 4, n, status)) continue;
      const float4 q = __ldg(x4 + v);
      f(q.x, 4 * v); f(q.y, 4 * v + 1); f(q.z, 4 * v + 2); f(q.w, 4 * v + 3);
    }
  } else {
    for (long long i = first; i < n; i += stride)
      if (TK_IN_BOUNDS(i, 1, n, status)) f(__ldg(x_row + i), i);
  }
}

template <bool Q4, bool MAG>
__global__ void __launch_bounds__(kLnThreads) tk_long_newton_kernel(const Problem P, const float zq, float* scratch) {
  __shared__ float sh[kLnThreads / 32 * 5];
  cg::grid_group grid = cg::this_grid();
  const int n = P.n, k = P.k;
  const float lam = P.lam, inv_lam = P.inv_lam, lam3 = P.lam3;
  constexpr float kTolRel = Q4 ? 1e-7f : 3e-7f;
  float* buf[2] = {scratch, scratch + (size_t)gridDim.x * kLnSlots};
  int phase = 0;
  int flags = 0;
  Math M = make_math(P);
  M.q4 = Q4; M.mag = MAG; M.gen = false;

  for (long long row = 0; row < P.rows; ++row) {
    const float* x_row = P.theta + row * (long long)n;
    float* o_row = P.out + row * (long long)n;
    NtRow S;
    nt_row_init(S, k);
    float wid = lam;
    // ---- start: moments of the keys (about the first key; phi even: about 0, and the keys above 0 counted)
    const float x0 = MAG ? 0.0f : __ldg(x_row);
    LnAcc a{0.f, 0.f, 0.f, 0u, 0u};
    bool bad = false;
    ln_for_each<MAG>(x_row, n, P.vec4, P.status, [&](float x, long long) {
      const float key = MAG ? fabsf(x) : x;
      const float dd = key - x0;
      a.v0 += dd; a.v1 = fmaf(dd, dd, a.v1);
      if (MAG) a.cnt += key > 0.0f;
      bad |= !(fabsf(x) < INFINITY);
    });
    a = ln_grid_sum(a, buf[phase & 1], sh, grid);
    ++phase;
    const float inv_n = 1.0f / (float)n;
    if (!MAG) {
      const float mean_d = a.v0 * inv_n;
      const float sd = sqrtf(fmaxf(a.v1 * inv_n - mean_d * mean_d, 0.0f));
      if (k == n) {
        S.piv = -FLT_MAX; S.off = -wid; S.done = true; S.noblock = true;
      } else {
        float tau0 = (x0 + mean_d) + zq * sd - (Q4 ? 0.75f : 0.5f) * lam;
        if (!(fabsf(tau0) < FLT_MAX)) tau0 = x0;
        S.piv = tau0;
      }
    } else {
      if (k == n || (long long)a.cnt < (long long)k) {
        S.piv = 0.0f; S.off = 0.0f; S.done = true; S.noblock = true;
      } else {
        const float t0 = zq * sqrtf(a.v1 * inv_n);
        float tau0 = Q4 ? t0 - 0.75f * lam * cbrtf(t0) : t0 / (1.0f + 0.5f * lam);
        if (!(tau0 > 0.0f && tau0 < FLT_MAX)) tau0 = 0.5f * t0;
        if (!(tau0 > 0.0f && tau0 < FLT_MAX)) tau0 = 1.0f;
        S.piv = tau0;
        S.lo_a = 0.0f; S.lo_o = -tau0;
      }
    }
    const bool early = S.done && S.noblock;

    // ---- the iteration (every thread of the grid holds the same S)
    int passes = 0;
#pragma unroll 1
    for (; passes < kNtMaxPasses && !S.done; ++passes) {
      if (MAG) wid = nt_width<Q4, true>(S.piv + S.off, lam);
      const float tol = kTolRel * (MAG ? fminf(wid, fmaxf(S.piv + S.off, 0.0f)) : wid);
      const float piv = S.piv, off = S.off;
      LnAcc c{0.f, 0.f, 0.f, 0u, 0u};
      ln_for_each<MAG>(x_row, n, P.vec4, P.status, [&](float x, long long) {
        const float t = ((MAG ? fabsf(x) : x) - piv) - off;
        const bool top = t >= wid, mid = t > 0.0f && !top;
        c.cnt2 += top; c.cnt += mid;
        const float tm = mid ? t : 0.0f;
        c.v0 += tm;
        if (Q4) { const float t2 = tm * tm; c.v1 += t2; c.v2 = fmaf(t2, tm, c.v2); }
      });
      c = ln_grid_sum(c, buf[phase & 1], sh, grid);
      ++phase;
      nt_step<Q4, MAG>(S, (int)c.cnt2, (int)c.cnt, c.v0, c.v1, c.v2, k, lam, lam3, wid, tol);
    }
    if (!S.done) { flags |= TK_FLAG_NOT_CONVERGED; S.a0 = k; S.b0 = k; }
    if (S.b0 <= S.a0) { S.a0 = k; S.b0 = k; }
    const bool block = S.b0 > S.a0;
    if (MAG) wid = nt_width<Q4, true>(S.piv + S.off, lam);

    // ---- row state (see tk_newton.cu: without a block any pivot between the (k+1)-th and the k-th key serves)
    float piv_state = S.piv, off_state = S.off;
    {
      const bool want_p = !block && !early;
      const bool safe = wid > 9.6e-7f * (fabsf(S.piv) + fabsf(S.off));
      if (want_p && !safe) {                   // uniform over the grid
        float cmin = INFINITY;
        const float piv = S.piv, off = S.off;
        ln_for_each<MAG>(x_row, n, P.vec4, P.status, [&](float x, long long) {
          const float key = MAG ? fabsf(x) : x;
          if ((key - piv) - off >= wid) cmin = fminf(cmin, key);
        });
        piv_state = ln_grid_min(cmin, buf[phase & 1], sh, grid);
        ++phase;
      }
      if (want_p && safe) piv_state = (S.piv + S.off) + 0.5f * wid;
      if (!block) off_state = 0.0f;
    }
    if (P.state_out && blockIdx.x == 0 && threadIdx.x == 0) {
      tk_rowstate st;
      st.pivot = piv_state; st.offset = off_state; st.a = S.a0; st.b = S.b0;
      P.state_out[row] = st;
    }

    // ---- dual map
    {
      const float piv = S.piv, off = S.off;
      const int mode = P.mode;
      auto y_of = [&](float x) -> float {
        const float t = ((MAG ? fabsf(x) : x) - piv) - off;
        if (!MAG) {
          const float a1 = __saturatef(t * inv_lam);
          const float y = Q4 ? a1 * a1 * a1 : a1;
          return mode == TK_TOPK ? y * x : y;
        }
        float v = 0.0f;
        if (t >= wid) v = M.vtop(fabsf(x));
        else if (t > 0.0f) v = M.rho(t);
        return signbit(x) ? -v : v;
      };
      const long long stride = (long long)gridDim.x * kLnThreads;
      const long long first = (long long)blockIdx.x * kLnThreads + threadIdx.x;
      if (P.vec4) {
        const float4* x4 = reinterpret_cast<const float4*>(x_row);
        float4* o4 = reinterpret_cast<float4*>(o_row);
        for (long long v = first; 4 * v < n; v += stride) {
          if (!TK_IN_BOUNDS(4 * v, 4, n, P.status)) continue;
          const float4 q = __ldg(x4 + v);
          o4[v] = make_float4(y_of(q.x), y_of(q.y), y_of(q.z), y_of(q.w));
        }
      } else {
        for (long long i = first; i < n; i += stride)
          if (TK_IN_BOUNDS(i, 1, n, P.status)) o_row[i] = y_of(__ldg(x_row + i));
      }
    }
    if (bad) flags |= TK_FLAG_NONFINITE;
  }
  if (flags && P.status) atomicOr(P.status, flags);
}

}  // namespace

float upper_normal_quantile(double tail);

// scratch the kernel needs: two buffers of one slot per block
size_t long_newton_scratch_bytes() { return 2 * (size_t)sm_count() * 8 * kLnSlots * sizeof(float); }

// Forward pass (p = 2 or 4/3, any mode, no permutation output) of a few rows of any length.  scratch:
// long_newton_scratch_bytes() of device memory, 16-byte aligned.
cudaError_t launch_long_newton(const Problem& P, void* scratch, cudaStream_t stream) {
  const bool q4 = P.q4 != 0, mag = P.mode == TK_TOPKMAG;
  const void* kern = q4 ? (mag ? (const void*)tk_long_newton_kernel<true, true> : (const void*)tk_long_newton_kernel<true, false>)
                        : (mag ? (const void*)tk_long_newton_kernel<false, true> : (const void*)tk_long_newton_kernel<false, false>);
  // all blocks must be resident at once: as many as fit, at most 8 per SM, and no more than the row gives work
  static int per_sm[64][4];
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  const int slot = (q4 ? 2 : 0) + (mag ? 1 : 0);
  int bps = (dev >= 0 && dev < 64) ? per_sm[dev][slot] : 0;
  if (bps == 0) {
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, kern, kLnThreads, 0);
    if (err != cudaSuccess) return err;
    if (bps < 1) return cudaErrorLaunchOutOfResources;
    if (bps > 8) bps = 8;
    if (dev >= 0 && dev < 64) per_sm[dev][slot] = bps;
  }
  long long blocks = (long long)sm_count() * bps;
  const long long useful = ((long long)P.n + 4 * kLnThreads - 1) / (4 * kLnThreads);
  if (blocks > useful) blocks = useful;
  if (blocks < 1) blocks = 1;
  const double tail = ((double)P.k - 0.5) / (double)P.n;
  float zq = upper_normal_quantile(mag ? 0.5 * tail : tail);
  Problem Pc = P;
  float* sc = static_cast<float*>(scratch);
  void* args[] = {(void*)&Pc, (void*)&zq, (void*)&sc};
  return cudaLaunchCooperativeKernel(kern, dim3((unsigned)blocks), dim3(kLnThreads), args, 0, stream);
}

}  // namespace tk
