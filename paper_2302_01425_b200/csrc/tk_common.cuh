// tk_common.cuh -- shared device helpers of the smoothed top-k kernels.
//
// Notation (Sec. 5 of the paper): s = keys in descending order, w = 1_k,
// h_i(v) = r*(s_i - v) + w_i phi(v), r*(t) = |t|^q / (q lambda^(q-1)),
// rho(t) = (r*)'(t) = sign(t) (|t|/lambda)^(q-1), q = p/(p-1) in {2, 4}.
// All arithmetic near the pooled block is done relative to the pivot
// c = k-th largest key: d_i = s_i - c, gamma = c + u.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "tk.h"

namespace tk {

enum What { W_FWD = 0, W_VJP = 1, W_ARGSORT = 2 };

constexpr int kLongTile = 4096;   // elements per thread block in the kernels for rows held in global memory

struct Problem {
  const float* theta;
  const float* gout;        // cotangent (VJP only)
  float* out;               // operator output (forward) or grad_theta (VJP)
  int32_t* perm_out;
  float* sorted_out;
  tk_rowstate* state_out;
  const tk_rowstate* state_in;
  int32_t* status;
  long long rows;
  int n, k;
  int N;                    // padded row length held on chip
  int q4;                   // 1: q = 4 (p = 4/3); 0: q = 2
  float qm1;                // q - 1 for any other q > 2 (sort-free solver and VJP from state only), else 0
  int mode;                 // tk_mode
  int what;                 // What
  int vec4;                 // rows may be accessed as float4
  float lam, inv_lam, lam3; // lambda, 1/lambda, lambda^3
  int sweeps;               // Dykstra path: number of sweeps, or their cap when tol > 0
  float tol;                // Dykstra path: > 0 = stop once no entry moved by more than this in a sweep
  int jvp;                  // tk_vjp_state kernels: the tangent goes through J instead of the cotangent through J^T
};

// ---------------------------------------------------------------- range-checked build
// With -DTK_DEBUG_BOUNDS (the second library target of build.py) the kernels of the default path test
// every global and shared index they form against the extent of its array: an index outside sets
// TK_FLAG_BOUNDS in the status word and the access is skipped -- no trap, the launch completes.  In the
// regular build the test is the constant true and costs nothing.
#ifdef TK_DEBUG_BOUNDS
__device__ __forceinline__ bool tk_bounds_ok(long long first, long long count, long long extent, int32_t* status) {
  const bool ok = first >= 0 && count >= 0 && first + count <= extent;
  if (!ok && status) atomicOr(status, TK_FLAG_BOUNDS);
  return ok;
}
#define TK_IN_BOUNDS(first, count, extent, status) \
  tk::tk_bounds_ok((long long)(first), (long long)(count), (long long)(extent), (status))
#else
#define TK_IN_BOUNDS(first, count, extent, status) true
#endif

// ---------------------------------------------------------------- host helpers
// Number of SMs of the current device, asked once per device (148, a B200, if the query fails).
inline int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    cached[dev] = v;
  }
  return cached[dev];
}

// ---------------------------------------------------------------- keys
// Order-preserving map float -> uint32 (larger float, larger integer).
__device__ __forceinline__ uint32_t f2key(float x) {
  uint32_t b = __float_as_uint(x);
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float key2f(uint32_t u) {
  uint32_t b = u ^ ((u >> 31) ? 0x80000000u : 0xFFFFFFFFu);
  return __uint_as_float(b);
}
// The sort key of an input: theta or |theta|, with -0 folded onto +0.
__device__ __forceinline__ float sort_key(float x, bool mag) {
  float k = mag ? fabsf(x) : x;
  return (k == 0.0f) ? 0.0f : k;
}

// ---------------------------------------------------------------- packed (key, index) elements
// Rows held on chip are sorted as 64-bit words (index < 65536):
// packed element: high word = order-preserving key, low word = (0xFFFF - index) << 1 | sign(theta).
// Larger packed value sorts first; equal keys sort by ascending index.
__device__ __forceinline__ unsigned long long pack(float x, int idx, bool mag, int n) {
  if (idx >= n) return (unsigned long long)(((0xFFFFu - (uint32_t)idx) << 1));  // padding sorts last
  uint32_t hi = f2key(sort_key(x, mag));
  uint32_t lo = ((0xFFFFu - (uint32_t)idx) << 1) | (__float_as_uint(x) >> 31);
  return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ float un_key(unsigned long long e) { return key2f((uint32_t)(e >> 32)); }
__device__ __forceinline__ int un_idx(unsigned long long e) {
  return 0xFFFF - (int)(((uint32_t)e >> 1) & 0xFFFFu);
}
__device__ __forceinline__ bool un_neg(unsigned long long e) { return ((uint32_t)e & 1u) != 0; }

// Branch-free compare-exchange and selection on packed elements.  Written as setp/selp so that
// the sorting networks compile to predicated selects (no divergent branches).
__device__ __forceinline__ void ce_desc(unsigned long long& a, unsigned long long& b) {   // a >= b after
  unsigned long long hi, lo;
  asm("{\n\t.reg .pred p;\n\tsetp.gt.u64 p, %2, %3;\n\tselp.b64 %0, %2, %3, p;\n\tselp.b64 %1, %3, %2, p;\n\t}"
      : "=l"(hi), "=l"(lo) : "l"(a), "l"(b));
  a = hi; b = lo;
}
// the larger (keepmax) or the smaller of r and o
__device__ __forceinline__ unsigned long long pick64(unsigned long long r, unsigned long long o, bool keepmax) {
  unsigned long long out;
  asm("{\n\t.reg .pred p, q;\n\tsetp.gt.u64 p, %2, %1;\n\tsetp.ne.u32 q, %3, 0;\n\txor.pred p, p, q;\n\t"
      "selp.b64 %0, %1, %2, p;\n\t}"
      : "=l"(out) : "l"(r), "l"(o), "r"((unsigned)keepmax));
  return out;
}
__device__ __forceinline__ unsigned long long sel64(bool c, unsigned long long x, unsigned long long y) {   // c ? x : y
  unsigned long long out;
  asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %3, 0;\n\tselp.b64 %0, %1, %2, p;\n\t}"
      : "=l"(out) : "l"(x), "l"(y), "r"((unsigned)c));
  return out;
}

// ---------------------------------------------------------------- scalar math
struct Math {
  float lam, inv_lam, lam3;
  float qm1;          // q - 1 when gen
  bool q4, mag;
  bool gen;           // q is neither 2 nor 4: rho(t) = (t/lam)^(q-1) through powf (t >= 0 here)

  __device__ __forceinline__ float rho(float t) const {
    float a = t * inv_lam;
    if (gen) return powf(a, qm1);
    return q4 ? a * a * a : a;
  }
  __device__ __forceinline__ float drho(float t) const {
    float a = t * inv_lam;
    if (gen) return qm1 * powf(a, qm1 - 1.0f) * inv_lam;
    return q4 ? 3.0f * a * a * inv_lam : inv_lam;
  }
  // z >= 0 with z^(q-1) + lam z = s (s >= 0): z = (s - v)/lam at the minimiser v of
  // h(v) = v^2/2 + r*(s - v), i.e. the point where rho(s - v) = v.  Newton from the right of the
  // root on a convex increasing function (q >= 3; for q < 3 it is concave and the same start is
  // left of the root after one step): monotone convergence.
  __device__ __forceinline__ float cubic_z(float s) const {
    if (!(s > 0.0f)) return 0.0f;
    if (gen) {
      float z = fminf(powf(s, 1.0f / qm1), s * inv_lam);
#pragma unroll 1
      for (int it = 0; it < 24; ++it) {
        const float zp = powf(z, qm1 - 1.0f);
        const float f = fmaf(zp + lam, z, -s);
        const float dz = f / fmaf(qm1, zp, lam);
        z = fmaxf(z - dz, 0.0f);
        if (fabsf(dz) <= 6e-8f * z) break;
      }
      return z;
    }
    float z = fminf(cbrtf(s), s * inv_lam);
#pragma unroll 1
    for (int it = 0; it < 16; ++it) {
      float f = fmaf(z * z + lam, z, -s);
      float dz = f / fmaf(3.0f * z, z, lam);
      z -= dz;
      if (fabsf(dz) <= 6e-8f * z) break;
    }
    return z;
  }
  // Minimiser of h_i for a rank < k (w_i = 1) singleton with key s.
  __device__ __forceinline__ float vtop(float s) const {
    if (!mag) return s - lam;
    if (!q4 && !gen) return s / (1.0f + lam);
    float z = cubic_z(s);
    float lz = lam * z;
    return (lz < 0.5f * s) ? s - lz : (gen ? powf(z, qm1) : z * z * z);
  }
  // Key distance above gamma = tau at which a rank < k element stops being
  // pooled: rho(width) = phi'(tau).
  __device__ __forceinline__ float width(float tau) const {
    if (!mag) return lam;
    float t = fmaxf(tau, 0.0f);
    if (gen) return lam * powf(t, 1.0f / qm1);
    return q4 ? lam * cbrtf(t) : lam * t;
  }
  // d/ds of the output of a top singleton (phi even): rho' / (rho' + 1).
  __device__ __forceinline__ float top_slope(float s) const {
    if (!mag) return 0.0f;
    if (!q4 && !gen) return 1.0f / (1.0f + lam);
    float z = cubic_z(s);              // z = (s - v)/lam, rho' = (q-1) z^(q-2) / lam
    float r = gen ? qm1 * powf(z, qm1 - 1.0f) * inv_lam : 3.0f * z * z * inv_lam;
    return r / (r + 1.0f);
  }
};

__device__ __forceinline__ Math make_math(const Problem& P) {
  Math m;
  m.lam = P.lam; m.inv_lam = P.inv_lam; m.lam3 = P.lam3;
  m.q4 = P.q4 != 0; m.mag = P.mode == TK_TOPKMAG;
  m.qm1 = P.qm1; m.gen = P.qm1 > 0.0f;
  return m;
}
// for the kernels that only ever see q = 2 or q = 4: the general branch folds away
__device__ __forceinline__ Math make_math_q24(const Problem& P) {
  Math m = make_math(P);
  m.gen = false;
  return m;
}

// Every later use of a row's solution classifies an element by its key alone:
// t = (key - pivot) - u, capped if t >= width(pivot + u), pooled if t > 0, else zero.  The solved
// u is rounded to fp32, and an element that sits a few 1e-9 inside the cap (a pooled rank whose
// rho is 1 - 1e-7) can then read as capped: harmless for the forward value, but the VJP of a
// capped element is a different formula.  This moves u by single ulps until the block's own edge
// ranks read as what the solve decided: a0-1 capped, a0 and b0-1 pooled, b0 zero.  A conflict
// (two edge keys closer than the arithmetic resolves) leaves u as it is.  key_at(i): sorted key of
// rank i, 0 <= i < n.
template <class KeyAt>
__device__ __forceinline__ float settle_offset(const Math& M, float piv, float u, int a0, int b0, int n,
                                               KeyAt key_at) {
  const float k_am1 = a0 > 0 ? key_at(a0 - 1) : INFINITY;
  const float k_a = key_at(a0), k_bm1 = key_at(b0 - 1);
  const float k_b = b0 < n ? key_at(b0) : -INFINITY;
#pragma unroll 1
  for (int it = 0; it < 8; ++it) {
    const float wid = M.width(piv + u);
    const bool up = ((k_a - piv) - u >= wid) || ((k_b - piv) - u > 0.0f);
    const bool down = !((k_bm1 - piv) - u > 0.0f) || ((k_am1 - piv) - u < wid);
    if (up == down) break;
    u = nextafterf(u, up ? INFINITY : -INFINITY);
  }
  return u;
}

// Root u of the pooled block's stationarity equation, from the block's power
// sums D_m = sum_B d_i^m (cnt members, m of them with w = 1), pivot c:
//   q = 2, phi = x   : sum (d_i - u)/lam = m            -> closed form
//   q = 2, phi even  : sum (d_i - u)/lam = m (c + u)    -> closed form (Sec. 5 example)
//   q = 4, phi = x   : sum (d_i - u)^3 = lam^3 m        (App. A.6 cubic)
//   q = 4, phi even  : sum (d_i - u)^3 = lam^3 m (c+u)
// The cubic is convex and decreasing in u left of the root; Newton from a point
// left of the root converges monotonically.  u_left must satisfy g(u_left) >= 0.
__device__ __forceinline__ double solve_block_u(bool q4, bool mag, double lam, double c, double cnt,
                                                double m, double D1, double D2, double D3,
                                                double u_left, int* not_converged) {
  if (!q4) {
    return mag ? (D1 - lam * m * c) / (cnt + lam * m) : (D1 - lam * m) / cnt;
  }
  const double l3m = lam * lam * lam * m;
  // Starting point: with mu = D1/cnt and central moments m2, m3 the equation is the depressed
  // cubic w^3 + P w + Q = 0 in w = u - mu, P >= 0, solved in fp32 by Cardano (stable form: the
  // two cube roots multiply to -P/3).  Newton in fp64 then needs a couple of steps; it is safe
  // from any start (a start right of the root steps to its left, then converges monotonically).
  double u = u_left;
  {
    const double mu = D1 / cnt;
    const double m2 = D2 - D1 * mu;
    const double m3 = D3 - 3.0 * mu * D2 + 2.0 * mu * mu * D1;
    const float Pc = (float)((3.0 * m2 + (mag ? l3m : 0.0)) / cnt);
    const float Qc = (float)((l3m * (mag ? (c + mu) : 1.0) - m3) / cnt);
    const float third = Pc * (1.0f / 3.0f);
    const float R = sqrtf(0.25f * Qc * Qc + third * third * third);
    // w = A + B with A = -sign(Q) cbrt(|Q|/2 + R), A B = -P/3 and A^3 + B^3 = -Q; written as
    // -Q / (A^2 - A B + B^2) it has no cancellation when the linear term dominates
    const float A = cbrtf(0.5f * fabsf(Qc) + R);
    const float B = (A != 0.0f) ? third / A : 0.0f;
    const float den = A * A + third + B * B;
    const float w = (den > 0.0f) ? -Qc / den : 0.0f;
    const double u0 = mu + (double)w;
    if (isfinite(u0)) u = u0;
  }
  bool ok = false;
#pragma unroll 1
  for (int it = 0; it < 64; ++it) {
    double g = ((-cnt * u + 3.0 * D1) * u - 3.0 * D2) * u + D3 - (mag ? l3m * (c + u) : l3m);
    double gp = -3.0 * ((cnt * u - 2.0 * D1) * u + D2) - (mag ? l3m : 0.0);
    if (!(gp < 0.0)) { ok = true; break; }
    double du = -g / gp;
    u += du;
    // phi = x: gamma enters through differences only, whose scale is lambda.  phi even: the
    // equation and the cap width depend on gamma = c + u itself, which can be far smaller.
    const double scale = mag ? fabs(c + u) : fabs(u) + lam;
    if (fabs(du) <= 1e-13 * scale + 1e-300) { ok = true; break; }
  }
  if (!ok && not_converged) *not_converged = 1;
  return u;
}

// ---------------------------------------------------------------- warp helpers
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace tk
