// tk_newton.cu -- the exact forward pass without a sort, for phi(x) = x (TK_MASK, TK_TOPK),
// p = 2 and p = 4/3, rows of up to 32768 elements held in registers.
//
// With w = 1_k the relaxed mask is the maximiser of <y, x> - R(y) over the capped simplex
// P(1_k) = {y in [0,1]^n, sum y = k} (Sec. 3), so y_i = clip(rho(x_i - tau), 0, 1) with tau the
// root of the non-increasing function
//   F(tau) = #{x_i - tau >= lambda} + sum_{0 < x_i - tau < lambda} rho(x_i - tau) - k.
// That root is the value gamma of the single pooled block pool-adjacent-violators ends with
// (Sec. 5), the elements strictly inside (gamma, gamma + lambda) are its members, those above it
// the top singletons.  F is piecewise linear (p = 2) or piecewise cubic (p = 4/3); on one piece
// it is the stationarity equation of that piece's candidate block (the example of Sec. 5, the
// cubic of App. A.6), solved here from the piece's power sums.  The iteration is Newton's on
// the pieces, inside a bracket that every evaluated point tightens:
//   - start: tau0 = mean + z std - lambda (1 - 1/q), z the normal quantile of 1 - k/n (a guess,
//     nothing depends on the data being Gaussian); for k <= 2 the k+1 largest keys are tracked
//     exactly instead, which gives the bracket (s_k - lambda, s_{k+1}) or "no block" at once;
//   - one pass over the registers classifies the row against tau (capped / inside / zero) and
//     sums t, t^2, t^3 over the inside keys; the piece's equation gives the next tau;
//   - a step that leaves the bracket is replaced by a step of doubling length towards the root,
//     then by bisection (of the ordered integer keys when the bracket spans many binades), and
//     after six Newton steps in a row one such step is forced: the loop ends;
//   - the root is accepted when a point reproduces the set of the pass before it and already
//     solves it to rounding, or when cm |du| is rounding-sized (F has slope >= 1/lambda until
//     it reaches an integer, so the root is then within that distance).
// tau is kept as pivot + offset, keys as d = x - pivot, so that t = d - offset is formed without
// cancellation; the row state stores exactly the pair the last pass classified with, and its
// counts, so the VJP from state sees the same classes.
//
// Layout: a row is held by G lanes of a warp (32/G rows per warp) or, above 2048 elements, by W whole
// warps, 64 keys per lane (fewer for rows of up to 32); the only exchange between the lanes of a
// row is the sum of the pass's counts and power sums (shuffles, plus one shared-memory slot per
// warp and a named barrier when W > 1).  Rows are read and written with coalesced 128-bit
// accesses straight from the registers; with one or two lanes per row through a shared-memory
// tile instead.
#include <float.h>
#include <stdlib.h>
#include <math.h>

#include "tk_newton_core.cuh"
#include "tk_team.cuh"

namespace tk {

// z with P(N(0,1) > z) = tail, by bisection on erfc (a starting guess for the iteration: 1e-6 is plenty)
float upper_normal_quantile(double tail) {
  double lo = -8.0, hi = 8.0;
  for (int i = 0; i < 28; ++i) {
    const double mid = 0.5 * (lo + hi);
    if (0.5 * erfc(mid * 0.70710678118654752440) > tail) lo = mid; else hi = mid;
  }
  return (float)(0.5 * (lo + hi));
}

namespace {

constexpr int kNtWarps = kTeamWarps;      // warps per thread block (more when a row takes more)

// rotation of the chunk order that makes the per-lane float4 reads of a quarter warp hit 8 bank groups
template <int E>
__device__ __forceinline__ int nt_rot(int lane) {
  constexpr int CH = E / 4;
  return CH >= 8 ? lane : (lane * CH) >> 3;
}

// keeps (m1 >= m2 >= m3) the three largest values seen
__device__ __forceinline__ void nt_top3(float x, float& m1, float& m2, float& m3) {
  float r = fminf(m1, x);
  m1 = fmaxf(m1, x);
  float r2 = fminf(m2, r);
  m2 = fmaxf(m2, r);
  m3 = fmaxf(m3, r2);
}

// threads per block, and the blocks per SM the register budget is set for: 24 warps of 80 registers with
// up to 32 keys per lane, 16 warps of 128 registers with 64
constexpr int nt_threads(int W) { return team_threads(W); }
// (p = 4/3 with two lanes per row through the staging tile keeps three more sums and the tile's addresses live: 20 warps of 102
// registers there, or the classification loop spills)
constexpr int nt_min_blocks(int E, int W, bool Q4 = false, bool STAGED = false, int G = 32) {
  return team_min_blocks(E >= 128 ? 8 : (E >= 64 ? 16 : ((Q4 && STAGED && E >= 32 && G == 2) ? 20 : 24)), W);
}

// ---------------------------------------------------------------- row access
// A row is spread over a team of T = G * W lanes (G lanes of one warp, or W whole warps), E keys per
// lane in E / 4 chunks of four.  DIRECT: chunk c of team lane tl is float4 number c * T + tl of the
// row, read from and written to global memory with coalesced 128-bit accesses (T * 16 contiguous
// bytes per row and instruction).  STAGED (one or two lanes per row, where that would be 16 or 32
// bytes): the warp's rows, contiguous in memory, go through a shared-memory tile with coalesced
// accesses, and every lane owns a contiguous span of the tile (chunk order rotated per lane: no
// bank conflicts).
template <int G, int E, int W, bool STAGED>
struct NtIO {
  static constexpr int CH = E / 4;
  static constexpr int T = G * W;
  const float* src;      // DIRECT: the row in global memory
  float* dst;
  float4* span4;         // STAGED: this lane's span of the tile
  int n, tl, rot, vec4, lane_in_warp;
  bool row_ok;
  long long first, extent;   // range-checked build: index of the row's first element in the tensor, its size
  int32_t* status;

  // STAGED: first word of this lane's span in the warp's tile
  __device__ __forceinline__ int tl_span() const { return lane_in_warp * E; }
  // index in the row of the first key of chunk c
  __device__ __forceinline__ int pos(int c) const {
    return STAGED ? tl * E + 4 * ((c + rot) & (CH - 1)) : 4 * (c * T + tl);
  }
  // the four words of chunk c as they are in memory (a chunk past the row re-reads the row's start:
  // no load depends on a test, so the loads of a lane are all in flight at once)
  __device__ __forceinline__ void load_raw(int c, float (&x)[4]) const {
    const int p0 = pos(c);
    if (STAGED) {
      const int slot = (c + rot) & (CH - 1);
      x[0] = x[1] = x[2] = x[3] = 0.0f;
      if (!TK_IN_BOUNDS(tl_span() + 4 * slot, 4, 32 * E, status)) return;
      const float4 v = span4[slot];
      x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else if (vec4) {
      const int pc = p0 < n ? p0 : 0;
      x[0] = x[1] = x[2] = x[3] = 0.0f;
      if (!TK_IN_BOUNDS(first + pc, 4, extent, status)) return;
      const float4 v = __ldg(reinterpret_cast<const float4*>(src + pc));
      x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pc = p0 + j < n ? p0 + j : 0;
        x[j] = TK_IN_BOUNDS(first + pc, 1, extent, status) ? __ldg(src + pc) : 0.0f;
      }
    }
  }
  // slots past the end of the row become -infinity, which never takes part.
  // ninf (may be null): set when a key of the row is itself -infinity
  __device__ __forceinline__ void mask(int c, float (&x)[4], bool* ninf = nullptr) const {
    const int p0 = pos(c);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool in = p0 + j < n;
      if (ninf && in && x[j] == -INFINITY) *ninf = true;
      if (!in) x[j] = -INFINITY;
    }
  }
  __device__ __forceinline__ void load(int c, float (&x)[4]) const {
    load_raw(c, x);
    mask(c, x);
  }
  __device__ __forceinline__ void store(int c, const float (&y)[4]) const {
    const int p0 = pos(c);
    if (STAGED) {
      const int slot = (c + rot) & (CH - 1);
      if (TK_IN_BOUNDS(tl_span() + 4 * slot, 4, 32 * E, status)) span4[slot] = make_float4(y[0], y[1], y[2], y[3]);
    } else if (vec4) {
      if (row_ok && p0 < n && TK_IN_BOUNDS(first + p0, 4, extent, status))
        *reinterpret_cast<float4*>(dst + p0) = make_float4(y[0], y[1], y[2], y[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (row_ok && p0 + j < n && TK_IN_BOUNDS(first + p0 + j, 1, extent, status)) dst[p0 + j] = y[j];
    }
  }
};

// One key against the window (t = key - tau): capped (t >= width), inside (0 < t < width) or zero.
// Counts and the inside keys' sums of t, t^2, t^3.
template <bool Q4>
__device__ __forceinline__ void nt_classify(float t, float wid, float& ct, float& cm, float& a, float& b, float& e) {
  // two compares, then adds under their predicates (written out so that no select is formed)
  if (!Q4) {
    asm("{\n\t.reg .pred ptop, pmid;\n\t"
        "setp.ge.f32 ptop, %3, %4;\n\t"
        "setp.gt.and.f32 pmid, %3, 0f00000000, !ptop;\n\t"
        "@ptop add.f32 %0, %0, 0f3F800000;\n\t"
        "@pmid add.f32 %1, %1, 0f3F800000;\n\t"
        "@pmid add.f32 %2, %2, %3;\n\t}"
        : "+f"(ct), "+f"(cm), "+f"(a)
        : "f"(t), "f"(wid));
  } else {
    asm("{\n\t.reg .pred ptop, pmid;\n\t.reg .f32 t2;\n\t"
        "setp.ge.f32 ptop, %5, %6;\n\t"
        "setp.gt.and.f32 pmid, %5, 0f00000000, !ptop;\n\t"
        "mul.f32 t2, %5, %5;\n\t"
        "@ptop add.f32 %0, %0, 0f3F800000;\n\t"
        "@pmid add.f32 %1, %1, 0f3F800000;\n\t"
        "@pmid add.f32 %2, %2, %5;\n\t"
        "@pmid add.f32 %3, %3, t2;\n\t"
        "@pmid fma.rn.f32 %4, t2, %5, %4;\n\t}"
        : "+f"(ct), "+f"(cm), "+f"(a), "+f"(b), "+f"(e)
        : "f"(t), "f"(wid));
  }
}

// Keeps the loads of later chunks behind this point: the second passes over a row (new pivot, top-k
// values, smallest capped key) run while the row's registers are live, and E more words in flight would spill.
__device__ __forceinline__ void nt_fence() { asm volatile("" ::: "memory"); }


// G lanes per row (W == 1) or W warps per row (G == 32), E keys per lane (E / 4 a power of two).
// KSEL: 0 = moment start, 1 / 2 = k is 1 / 2 (W == 1, phi = x only).  MAG: phi(x) = x^2/2, keys |theta|.
template <int G, int E, int W, bool Q4, int KSEL, bool STAGED, bool MAG>
__global__ void __launch_bounds__(nt_threads(W), nt_min_blocks(E, W, Q4, STAGED, G)) tk_newton_kernel(const Problem P, const float zq, const int pf_rows) {
  extern __shared__ float4 nt_smem4[];
  static_assert(W == 1 || G == 32, "several warps per row: every lane of them belongs to the row");
  static_assert(!STAGED || W == 1, "the staging tile belongs to one warp");
  static_assert(!MAG || KSEL == 0, "the magnitude mode starts from the moments");
  constexpr int BW = kNtWarps > W ? kNtWarps : W;   // warps per block
  constexpr int TEAMS = BW / W;                      // teams (of W warps) per block
  constexpr int R = W > 1 ? 1 : 32 / G;              // rows per team
  constexpr int CH = E / 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int team = warp / W, wit = warp % W;
  const long long row0 = ((long long)blockIdx.x * TEAMS + team) * R;
  if (row0 >= P.rows) return;                  // the whole team
  const int n = P.n, k = P.k;
  const int rl = lane / G, lig = lane % G;
  const long long row = row0 + rl;
  const bool row_ok = row < P.rows;
  const float lam = P.lam, inv_lam = P.inv_lam, lam3 = P.lam3;
  float wid = P.lam;                           // phi = x: constant; phi even: follows tau
  constexpr float kTolRel = Q4 ? 1e-7f : 3e-7f;
  float* smem = reinterpret_cast<float*>(nt_smem4);
  // shared memory: [STAGED: one tile of 32 E floats per warp] [W > 1: two buffers of W * 4 words per team]
  float* red = smem + (STAGED ? BW * 32 * E : 0) + team * (2 * W * 4);
  const int bar = 1 + team;
  int phase = 0;                               // which of the two buffers the next team sum uses

  NtIO<G, E, W, STAGED> io;
  io.n = n; io.vec4 = P.vec4; io.row_ok = row_ok;
  io.tl = W > 1 ? wit * 32 + lane : lig;
  io.rot = nt_rot<E>(lane);
  // a group past the last row works on the last row again and stores nothing
  const long long row_c = row_ok ? row : P.rows - 1;
  io.src = P.theta + row_c * (long long)n;
  io.dst = P.out + row_c * (long long)n;
  io.first = row_c * (long long)n; io.extent = P.rows * (long long)n; io.status = P.status;
  io.lane_in_warp = lane;
  io.span4 = nullptr;
  if (STAGED) {
    // ---- stage the warp's rows (contiguous in memory) in its tile, row stride G * E
    constexpr int RS = G * E;
    float* tile = smem + warp * (32 * E);
    io.span4 = reinterpret_cast<float4*>(tile + lane * E);
    const int rows_here = (int)(P.rows - row0 < (long long)R ? P.rows - row0 : (long long)R);
    const float* src = P.theta + row0 * (long long)n;
    if (n == RS) {
      const int total = rows_here * n;
      if (P.vec4) {
        const float4* s4 = reinterpret_cast<const float4*>(src);
        float4* t4 = reinterpret_cast<float4*>(tile);
        for (int v = lane; 4 * v < total; v += 32)
          if (TK_IN_BOUNDS(row0 * (long long)n + 4 * v, 4, io.extent, P.status) && TK_IN_BOUNDS(4 * v, 4, 32 * E, P.status)) t4[v] = __ldg(s4 + v);
      } else {
        for (int i = lane; i < total; i += 32)
          if (TK_IN_BOUNDS(row0 * (long long)n + i, 1, io.extent, P.status) && TK_IN_BOUNDS(i, 1, 32 * E, P.status)) tile[i] = __ldg(src + i);
      }
    } else {
      for (int r = 0; r < rows_here; ++r) {
        if (P.vec4) {
          const float4* s4 = reinterpret_cast<const float4*>(src + (long long)r * n);
          float4* t4 = reinterpret_cast<float4*>(tile + r * RS);
          for (int v = lane; 4 * v < n; v += 32)
            if (TK_IN_BOUNDS((row0 + r) * (long long)n + 4 * v, 4, io.extent, P.status) && TK_IN_BOUNDS(r * RS + 4 * v, 4, 32 * E, P.status)) t4[v] = __ldg(s4 + v);
        } else {
          for (int i = lane; i < n; i += 32)
            if (TK_IN_BOUNDS((row0 + r) * (long long)n + i, 1, io.extent, P.status) && TK_IN_BOUNDS(r * RS + i, 1, 32 * E, P.status)) tile[r * RS + i] = __ldg(src + (long long)r * n + i);
        }
      }
    }
    // lanes whose row lies past the last one solve a row of zeros and store nothing
    for (int i = rows_here * RS + lane; i < R * RS; i += 32)
      if (TK_IN_BOUNDS(i, 1, 32 * E, P.status)) tile[i] = 0.0f;
    __syncwarp();
  }

  float d[E];
  bool bad = false;                            // a NaN or an infinity among this lane's keys
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    float x4[4];
    io.load_raw(c, x4);
#pragma unroll
    for (int j = 0; j < 4; ++j) d[4 * c + j] = MAG ? fabsf(x4[j]) : x4[j];
  }
  // a row that fills its lanes exactly has no slot to mark (and a -infinity in it shows in the sums below)
  const bool full = n == (STAGED ? G : G * W) * E;
  if (!full) {
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      float x4[4] = {d[4 * c], d[4 * c + 1], d[4 * c + 2], d[4 * c + 3]};
      io.mask(c, x4, &bad);
      d[4 * c] = x4[0]; d[4 * c + 1] = x4[1]; d[4 * c + 2] = x4[2]; d[4 * c + 3] = x4[3];
    }
  }

  // ---- start: bracket and first tau
  NtRow S;
  nt_row_init(S, k);
  float lo = -FLT_MAX, hi = FLT_MAX;
  if (KSEL == 0) {
    // sums about the row's first key: mean and spread of the keys
    const float x0 = MAG ? 0.0f : __ldg(io.src);
    float v[2] = {0.f, 0.f};
    uint32_t nnz = 0;                          // phi even: keys above 0
    if (full) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float dd = d[i] - x0;
        v[0] += dd; v[1] = fmaf(dd, dd, v[1]);
      }
    } else {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float dd = (d[i] == -INFINITY) ? 0.0f : d[i] - x0;
        v[0] += dd; v[1] = fmaf(dd, dd, v[1]);
      }
    }
    if (MAG) {
#pragma unroll
      for (int i = 0; i < E; ++i) nnz += d[i] > 0.0f;
    }
    team_allsum<G, W, 2>(v, nnz, red + (phase & 1) * (W * 4), wit, lane, bar);
    ++phase;
    if (!(v[1] < INFINITY)) {                  // overflow, an infinity or a NaN: look at the keys themselves
#pragma unroll
      for (int i = 0; i < E; ++i) bad |= !(fabsf(d[i]) < INFINITY) && (full || d[i] != -INFINITY);
    }
    const float inv_n = 1.0f / (float)n;
    const float mean_d = v[0] * inv_n;
    const float sd = sqrtf(fmaxf(v[1] * inv_n - mean_d * mean_d, 0.0f));
    if (!MAG) {
      if (k == n) {                            // everything is selected
        S.piv = -FLT_MAX; S.off = -wid; S.done = true; S.noblock = true;
      } else {
        float tau0 = (x0 + mean_d) + zq * sd - (Q4 ? 0.75f : 0.5f) * lam;
        if (!(fabsf(tau0) < FLT_MAX)) tau0 = x0;
        S.piv = tau0;
      }
    } else {
      if (k == n || (int)nnz < k) {
        // the k-th largest |theta| is 0 (or everything is selected): every key is a top singleton
        S.piv = 0.0f; S.off = 0.0f; S.done = true; S.noblock = true;
      } else {
        // zq: the upper k/(2n) quantile of N(0,1); the keys of a zero-mean row are its absolute values.
        // About k keys lie above gamma + width/2 (q = 2) or gamma + 3 width/4 (q = 4).
        const float t0 = zq * sqrtf(v[1] * inv_n);
        float tau0 = Q4 ? t0 - 0.75f * lam * cbrtf(t0) : t0 / (1.0f + 0.5f * lam);
        if (!(tau0 > 0.0f && tau0 < FLT_MAX)) tau0 = 0.5f * t0;
        if (!(tau0 > 0.0f && tau0 < FLT_MAX)) tau0 = 1.0f;
        S.piv = tau0;
        lo = 0.0f; S.lo_o = -tau0;             // F(0) = n - k >= 0: every key is capped at tau = 0
      }
    }
  } else {
    float m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY, fin = 0.0f;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      nt_top3(d[i], m1, m2, m3);
      fin = fmaf((!full && d[i] == -INFINITY) ? 0.0f : d[i], 0.0f, fin);
    }
    bad |= fin != fin;
#pragma unroll
    for (int o = G >> 1; o > 0; o >>= 1) {
      const float p1 = __shfl_xor_sync(0xffffffffu, m1, o), p2 = __shfl_xor_sync(0xffffffffu, m2, o),
                  p3 = __shfl_xor_sync(0xffffffffu, m3, o);
      nt_top3(p1, m1, m2, m3); nt_top3(p2, m1, m2, m3); nt_top3(p3, m1, m2, m3);
    }
    const float c = KSEL == 1 ? m1 : m2, sk = KSEL == 1 ? m2 : m3;   // k-th and (k+1)-th largest key
    // The bracket (s_k - lambda, s_{k+1}) is kept relative to the pivot s_{k+1}: the gap s_k - s_{k+1}
    // is exact there, and so is the end s_k - lambda the root may sit a hair inside of.
    const float dc = c - sk;
    lo = c - wid; hi = sk;
    if (!(dc < wid)) {                         // vtop(s_k) >= s_{k+1}: no violation, no block
      S.piv = c; S.off = -wid; S.done = true; S.noblock = true;
    } else {
      S.piv = sk; S.lo_o = dc - wid; S.hi_o = 0.0f; S.off = 0.5f * S.lo_o;
    }
  }
  const bool early = S.done && S.noblock;      // pivot already exact
  S.lo_a = lo; S.hi_a = hi;
#pragma unroll
  for (int i = 0; i < E; ++i) d[i] -= S.piv;

  // The rows this SM slot will hold one wave of blocks from now are asked into L2 once this wave's
  // own keys have arrived: HBM keeps streaming while the warps iterate on their registers.  One 128-byte
  // line per lane covers the team's E * T keys.
  if (!STAGED) {
    const long long prow = row + pf_rows;
    const int line = (W > 1 ? wit * 32 + lane : lig) * 32;            // first key of this lane's line
    if (pf_rows > 0 && prow < P.rows && line < n)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(P.theta + prow * (long long)n + line));
  } else {
    const long long prow0 = row0 + pf_rows;                            // the warp's rows are contiguous
    const long long first = prow0 * (long long)n + lane * 32, end = P.rows * (long long)n;
    if (pf_rows > 0 && first < end && lane * 32 < R * n)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(P.theta + first));
  }

  // ---- the iteration
  int passes = 0;
#pragma unroll 1
  for (; passes < kNtMaxPasses; ++passes) {
    if (__all_sync(0xffffffffu, S.done)) break;
    if (MAG) wid = nt_width<Q4, true>(S.piv + S.off, lam);
    // phi even: tau enters the width and the piece's equation itself, so a step is small against tau too
    const float tol = kTolRel * (MAG ? fminf(wid, fmaxf(S.piv + S.off, 0.0f)) : wid);
    // Counts are kept as floats (exact: a lane holds at most E keys) and every update is an add under a
    // predicate: two compares per key on the ALU pipe, everything else on the FMA pipe.
    float ct0 = 0.f, ct1 = 0.f, cm0 = 0.f, cm1 = 0.f;
    float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, e0 = 0.f, e1 = 0.f;
    const float off = S.off;
#pragma unroll
    for (int i = 0; i < E; i += 2) {
      nt_classify<Q4>(d[i] - off, wid, ct0, cm0, a0, b0, e0);
      nt_classify<Q4>(d[i + 1] - off, wid, ct1, cm1, a1, b1, e1);
    }
    float v[Q4 ? 3 : 1];
    v[0] = a0 + a1;
    if (Q4) { v[1] = b0 + b1; v[2] = e0 + e1; }
    uint32_t packed = (uint32_t)(int)(ct0 + ct1) | ((uint32_t)(int)(cm0 + cm1) << 16);
    team_allsum<G, W, Q4 ? 3 : 1>(v, packed, red + (phase & 1) * (W * 4), wit, lane, bar);
    ++phase;
    if (!S.done) {
      nt_step<Q4, MAG>(S, (int)(packed & 0xffffu), (int)(packed >> 16), v[0], Q4 ? v[1] : 0.0f,
                       Q4 ? v[Q4 ? 2 : 0] : 0.0f, k, lam, lam3, wid, tol);
      if (S.repiv) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          float x4[4];
          io.load(c, x4);
#pragma unroll
          for (int j = 0; j < 4; ++j)      // (a slot past the row stays at -infinity)
            d[4 * c + j] = ((MAG && x4[j] != -INFINITY) ? fabsf(x4[j]) : x4[j]) - S.piv;
          if ((c & 3) == 3) nt_fence();
        }
      }
    }
  }
  int flags = 0;
  if (!S.done) {                               // cap reached: keep the last point, say so
    flags |= TK_FLAG_NOT_CONVERGED;
    S.a0 = k; S.b0 = k;
  }
  if (S.b0 <= S.a0) { S.a0 = k; S.b0 = k; }
  const bool block = S.b0 > S.a0;
  if (MAG) wid = nt_width<Q4, true>(S.piv + S.off, lam);   // of the point the last pass classified at

  // ---- row state.  Without a block the VJP classifies by key >= pivot: any value above the
  // (k+1)-th largest key and not above the k-th serves; tau + lambda/2 is one when lambda is
  // resolved at the keys' magnitude, else the smallest capped key is looked up.
  float piv_state = S.piv, off_state = S.off;
  {
    const bool want_p = row_ok && !block && !early;
    const bool safe = wid > 9.6e-7f * (fabsf(S.piv) + fabsf(S.off));
    const bool scan = want_p && !safe;
    if (__any_sync(0xffffffffu, scan)) {       // uniform over the warps of a row: they hold the same S
      float cmin = INFINITY;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        float x4[4];
        io.load(c, x4);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (d[4 * c + j] - S.off >= wid) cmin = fminf(cmin, MAG ? fabsf(x4[j]) : x4[j]);
        if ((c & 3) == 3) nt_fence();
      }
      cmin = team_gmin<G>(cmin);
      if (W > 1) {
        float* rb = red + (phase & 1) * (W * 4);
        ++phase;
        if (lane == 0 && TK_IN_BOUNDS(team * (2 * W * 4) + ((phase - 1) & 1) * (W * 4) + wit * 4, 1, TEAMS * 2 * W * 4, P.status)) rb[wit * 4] = cmin;
        team_barrier(bar, W * 32);
        cmin = rb[0];
#pragma unroll
        for (int w = 1; w < W; ++w) cmin = fminf(cmin, rb[w * 4]);
      }
      if (scan) piv_state = cmin;
    }
    if (want_p && safe) piv_state = (S.piv + S.off) + 0.5f * wid;
    if (!block) off_state = 0.0f;
  }
  if (P.state_out && row_ok && lig == 0 && wit == 0 && TK_IN_BOUNDS(row, 1, P.rows, P.status)) {
    tk_rowstate st;
    st.pivot = piv_state; st.offset = off_state; st.a = S.a0; st.b = S.b0;
    P.state_out[row] = st;
  }

  // ---- dual map y = rho(clamp(key - tau)), in the order the keys were read.  phi even: a top singleton
  // is its own minimiser vtop(key) (stationarity rho(key - v) = v), and the sign of theta comes back
  if (!MAG) {
    const float shift = -S.off * inv_lam;
    const bool times_x = P.mode == TK_TOPK;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      float y[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a = __saturatef(fmaf(d[4 * c + j], inv_lam, shift));
        y[j] = Q4 ? a * a * a : a;
      }
      if (times_x) {
        float x4[4];
        io.load(c, x4);
#pragma unroll
        for (int j = 0; j < 4; ++j) y[j] = (x4[j] == -INFINITY) ? 0.0f : y[j] * x4[j];
      }
      io.store(c, y);
      if (times_x && (c & 3) == 3) nt_fence();
    }
  } else {
    Math M = make_math(P);
    M.q4 = Q4; M.mag = true; M.gen = false;
    const float off = S.off;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      float x4[4], y[4];
      io.load(c, x4);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float t = d[4 * c + j] - off;
        float v = 0.0f;
        if (t >= wid) v = M.vtop(fabsf(x4[j]));
        else if (t > 0.0f) v = M.rho(t);
        y[j] = signbit(x4[j]) ? -v : v;
      }
      io.store(c, y);
      if ((c & 3) == 3) nt_fence();
    }
  }
  if (STAGED) {
    constexpr int RS = G * E;
    __syncwarp();
    const float* tile = smem + warp * (32 * E);
    const int rows_here = (int)(P.rows - row0 < (long long)R ? P.rows - row0 : (long long)R);
    float* dst = P.out + row0 * (long long)n;
    if (n == RS) {
      const int total = rows_here * n;
      if (P.vec4) {
        float4* d4 = reinterpret_cast<float4*>(dst);
        const float4* t4 = reinterpret_cast<const float4*>(tile);
        for (int v = lane; 4 * v < total; v += 32)
          if (TK_IN_BOUNDS(row0 * (long long)n + 4 * v, 4, io.extent, P.status) && TK_IN_BOUNDS(4 * v, 4, 32 * E, P.status)) d4[v] = t4[v];
      } else {
        for (int i = lane; i < total; i += 32)
          if (TK_IN_BOUNDS(row0 * (long long)n + i, 1, io.extent, P.status) && TK_IN_BOUNDS(i, 1, 32 * E, P.status)) dst[i] = tile[i];
      }
    } else {
      for (int r = 0; r < rows_here; ++r) {
        if (P.vec4) {
          float4* d4 = reinterpret_cast<float4*>(dst + (long long)r * n);
          const float4* t4 = reinterpret_cast<const float4*>(tile + r * RS);
          for (int v = lane; 4 * v < n; v += 32)
            if (TK_IN_BOUNDS((row0 + r) * (long long)n + 4 * v, 4, io.extent, P.status) && TK_IN_BOUNDS(r * RS + 4 * v, 4, 32 * E, P.status)) d4[v] = t4[v];
        } else {
          for (int i = lane; i < n; i += 32)
            if (TK_IN_BOUNDS((row0 + r) * (long long)n + i, 1, io.extent, P.status) && TK_IN_BOUNDS(r * RS + i, 1, 32 * E, P.status)) dst[(long long)r * n + i] = tile[r * RS + i];
        }
      }
    }
  }
  if (P.status) {
    if (bad) flags |= TK_FLAG_NONFINITE;
    if (flags) atomicOr(P.status, flags);
  }
}

template <int G, int E, int W, bool Q4, int KSEL, bool STAGED, bool MAG>
cudaError_t nt_launch(const Problem& P, float zq, cudaStream_t stream) {
  static const bool no_pf = getenv("TK_NT_NOPF") != nullptr;
  constexpr int BW = kNtWarps > W ? kNtWarps : W;
  constexpr int TEAMS = BW / W;
  constexpr int smem = (STAGED ? BW * 32 * E * (int)sizeof(float) : 0) + (W > 1 ? TEAMS * 2 * W * 4 * (int)sizeof(float) : 0);
  auto kern = tk_newton_kernel<G, E, W, Q4, KSEL, STAGED, MAG>;
  if (smem > 48 * 1024) {
    static bool configured[64];
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (err != cudaSuccess) return err;
      if (dev >= 0 && dev < 64) configured[dev] = true;
    }
  }
  constexpr long long rows_per_block = (long long)TEAMS * (W > 1 ? 1 : 32 / G);
  const unsigned blocks = (unsigned)((P.rows + rows_per_block - 1) / rows_per_block);
  // rows in flight on the whole GPU: the distance the prefetch looks ahead
  const long long wave = (long long)sm_count() * nt_min_blocks(E, W, Q4, STAGED, G) * rows_per_block;
  const int pf_rows = no_pf ? 0 : (int)(wave < 0x7fffffff ? wave : 0);
  kern<<<blocks, BW * 32, smem, stream>>>(P, zq, pf_rows);
  return cudaGetLastError();
}

// KS: the shape also has the variants that track the k + 1 largest keys (k <= 2, phi = x)
template <int G, int E, int W, bool KS, bool STAGED>
cudaError_t nt_launch_q(const Problem& P, float zq, cudaStream_t stream) {
  const bool q4 = P.q4 != 0;
  if (P.mode == TK_TOPKMAG)
    return q4 ? nt_launch<G, E, W, true, 0, STAGED, true>(P, zq, stream)
              : nt_launch<G, E, W, false, 0, STAGED, true>(P, zq, stream);
  if (KS && P.k == 1)
    return q4 ? nt_launch<G, E, W, true, KS ? 1 : 0, STAGED, false>(P, zq, stream)
              : nt_launch<G, E, W, false, KS ? 1 : 0, STAGED, false>(P, zq, stream);
  if (KS && P.k == 2)
    return q4 ? nt_launch<G, E, W, true, KS ? 2 : 0, STAGED, false>(P, zq, stream)
              : nt_launch<G, E, W, false, KS ? 2 : 0, STAGED, false>(P, zq, stream);
  return q4 ? nt_launch<G, E, W, true, 0, STAGED, false>(P, zq, stream)
            : nt_launch<G, E, W, false, 0, STAGED, false>(P, zq, stream);
}

}  // namespace

int newton_max_n() { return 32768; }

// Forward pass with p = 2 or 4/3, rows of up to newton_max_n() elements, no permutation output.
cudaError_t launch_newton(const Problem& P, cudaStream_t stream) {
  const int n = P.n;
  // phi even: the keys are absolute values, k of n lie above the upper k/(2n) quantile of a zero-mean row
  const double tail = ((double)P.k - 0.5) / (double)n;
  const float zq = upper_normal_quantile(P.mode == TK_TOPKMAG ? 0.5 * tail : tail);
  // 32 keys per lane (more lanes per row and more rows in flight beat longer register rows); one or
  // two lanes per row go through the staging tile
  if (n <= 8) return nt_launch_q<1, 8, 1, true, true>(P, zq, stream);
  if (n <= 16) return nt_launch_q<1, 16, 1, true, true>(P, zq, stream);
  if (n <= 32) return nt_launch_q<1, 32, 1, true, true>(P, zq, stream);
  if (n <= 64) {
    // a router-sized batch leaves the SMs short of warps at 16 rows per warp: 8 rows per warp then
    if (P.rows < (long long)sm_count() * 24 * 16) return nt_launch_q<4, 16, 1, true, false>(P, zq, stream);
    return nt_launch_q<2, 32, 1, true, true>(P, zq, stream);
  }
  if (n <= 128) return nt_launch_q<4, 32, 1, true, false>(P, zq, stream);
  if (n <= 256) return nt_launch_q<8, 32, 1, false, false>(P, zq, stream);
  if (n <= 512) return nt_launch_q<16, 32, 1, false, false>(P, zq, stream);
  if (n <= 1024) return nt_launch_q<32, 32, 1, false, false>(P, zq, stream);
  if (n <= 2048) return nt_launch_q<32, 32, 2, false, false>(P, zq, stream);
  if (n <= 4096) return nt_launch_q<32, 32, 4, false, false>(P, zq, stream);
  if (n <= 8192) return nt_launch_q<32, 32, 8, false, false>(P, zq, stream);
  if (n <= 16384) return nt_launch_q<32, 32, 16, false, false>(P, zq, stream);
  return nt_launch_q<32, 64, 16, false, false>(P, zq, stream);
}

}  // namespace tk
