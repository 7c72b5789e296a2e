// tk_long.cu -- rows too long to hold on chip (n > 16384).
//
//   1. segmented stable LSD radix sort of (key, index) in global memory: four
//      8-bit passes, each = digit histogram per tile -> exclusive scan per row
//      -> stable scatter.  Keys are the bit-inverted order-preserving integers,
//      so the ascending radix order is the descending key order and equal keys
//      keep their ascending original index (Sec. 3, argsort).
//   2. prefix sums of d, d^2, d^3 (d = key - pivot) over the poolable window,
//      per tile in fp32 plus fp64 tile offsets.
//   3. one thread block per row searches the single pooled block [a, b) with
//      the same monotone predicates as the on-chip kernels, then sums the block
//      directly and solves its stationarity equation (Sec. 5, App. A.6).
//   4. dual map in sorted coordinates and scatter to the original positions
//      (Prop. 2, Prop. 5/6).
//
// All scratch lives in the caller's workspace; every launch is on the caller's
// stream; nothing waits on another thread block (separate launches instead).
#include "tk_common.cuh"

namespace tk {

namespace {

constexpr int TILE = kLongTile;     // elements per thread block in the sort and scan kernels
constexpr int TPB = 256;            // threads per block there
constexpr int IPT = TILE / TPB;     // 16 elements per thread
constexpr int WARPS = TPB / 32;
constexpr int WCHUNK = TILE / WARPS;   // 512 consecutive elements per warp in the scatter kernel
constexpr int RADIX = 256;

struct LongWs {
  uint32_t* keyA; uint32_t* keyB;
  int32_t* idxA; int32_t* idxB;
  uint32_t* hist;        // [rows][RADIX][tiles]
  uint32_t* dtot;        // [rows][RADIX] digit totals (rows with many tiles)
  float* pin1; float* pin2; float* pin3;   // in-tile exclusive prefix of d, d^2, d^3 (window only)
  double* tsum;          // [rows][3][tiles] tile totals, turned into exclusive offsets
  tk_rowstate* state;    // [rows] when the caller passes none
};

__host__ __device__ inline size_t align_up(size_t x) { return (x + 255) & ~size_t(255); }

// sort key of pass 0 read from theta: ascending radix on ~f2key == descending key
__device__ __forceinline__ uint32_t radix_key(float x, bool mag) { return ~f2key(sort_key(x, mag)); }
__device__ __forceinline__ float radix_key_to_float(uint32_t rk) { return key2f(~rk); }

// ---- pass kernels -------------------------------------------------------------
template <bool FIRST>
__global__ void __launch_bounds__(TPB) long_hist_kernel(const float* theta, const uint32_t* keys_in,
                                                        uint32_t* hist, int n, int tiles, int shift, int mag,
                                                        int32_t* status) {
  __shared__ uint32_t h[RADIX];
  const int tile = blockIdx.x;
  const long long row = blockIdx.y;
  for (int i = threadIdx.x; i < RADIX; i += TPB) h[i] = 0;
  __syncthreads();
  const long long base = row * (long long)n;
  const int start = tile * TILE;
#pragma unroll 4
  for (int i = 0; i < IPT; ++i) {
    int pos = start + i * TPB + threadIdx.x;
    if (pos < n) {
      uint32_t key;
      if (FIRST) {
        const float x = __ldg(theta + base + pos);
        if (!isfinite(x) && status) atomicOr(status, TK_FLAG_NONFINITE);
        key = radix_key(x, mag != 0);
      } else {
        key = keys_in[base + pos];
      }
      atomicAdd(&h[(key >> shift) & 0xFF], 1u);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < RADIX; i += TPB)
    hist[(row * RADIX + i) * (long long)tiles + tile] = h[i];
}

// exclusive scan of hist[row][digit][tile] in (digit, tile) order: one block per row.  Each warp
// owns digits w, w + 32, ..: it sums a digit's tiles with coalesced reads, the 256 digit totals
// are scanned by the first warps, then each warp scans its digits' tiles 32 at a time.
__global__ void __launch_bounds__(1024) long_scan_hist_kernel(uint32_t* hist, int tiles) {
  __shared__ uint32_t dtot[RADIX];
  const long long row = blockIdx.x;
  uint32_t* h = hist + row * (long long)RADIX * tiles;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int d = warp; d < RADIX; d += 32) {
    const uint32_t* hd = h + (long long)d * tiles;
    uint32_t s = 0;
    for (int i = lane; i < tiles; i += 32) s += hd[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) dtot[d] = s;
  }
  __syncthreads();
  if (warp == 0) {      // exclusive scan of the 256 digit totals, 8 per lane
    uint32_t v[8], s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[i] = dtot[lane * 8 + i]; s += v[i]; }
    uint32_t inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
    uint32_t run = inc - s;
#pragma unroll
    for (int i = 0; i < 8; ++i) { dtot[lane * 8 + i] = run; run += v[i]; }
  }
  __syncthreads();
  for (int d = warp; d < RADIX; d += 32) {
    uint32_t* hd = h + (long long)d * tiles;
    uint32_t carry = dtot[d];
    for (int i0 = 0; i0 < tiles; i0 += 32) {
      const int i = i0 + lane;
      const uint32_t v = (i < tiles) ? hd[i] : 0u;
      uint32_t inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { uint32_t up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
      if (i < tiles) hd[i] = carry + inc - v;
      carry += __shfl_sync(0xffffffffu, inc, 31);
    }
  }
}

// The same scan for rows with many tiles, spread over 256 blocks per row: digit totals first,
// then every block derives its digit's base from the totals and scans its own tiles.
__global__ void __launch_bounds__(256) long_digit_total_kernel(const uint32_t* hist, uint32_t* dtot, int tiles) {
  __shared__ uint32_t red[8];
  const int d = blockIdx.x;
  const long long row = blockIdx.y;
  const uint32_t* hd = hist + (row * RADIX + d) * (long long)tiles;
  uint32_t s = 0;
  for (int i = threadIdx.x; i < tiles; i += 256) s += hd[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t tot = 0;
    for (int w = 0; w < 8; ++w) tot += red[w];
    dtot[row * RADIX + d] = tot;
  }
}

__global__ void __launch_bounds__(256) long_digit_scan_kernel(uint32_t* hist, const uint32_t* dtot, int tiles) {
  __shared__ uint32_t red[8];
  __shared__ uint32_t wsum[8];
  const int d = blockIdx.x;
  const long long row = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // base of this digit: sum of the totals of the smaller digits
  uint32_t b = (threadIdx.x < d) ? dtot[row * RADIX + threadIdx.x] : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) b += __shfl_xor_sync(0xffffffffu, b, o);
  if (lane == 0) red[warp] = b;
  __syncthreads();
  uint32_t carry = 0;
  for (int w = 0; w < 8; ++w) carry += red[w];
  uint32_t* hd = hist + (row * RADIX + d) * (long long)tiles;
  for (int i0 = 0; i0 < tiles; i0 += 256) {
    const int i = i0 + threadIdx.x;
    const uint32_t v = (i < tiles) ? hd[i] : 0u;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
    __syncthreads();                       // wsum of the previous chunk has been read
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    uint32_t woff = 0, tot = 0;
    for (int w = 0; w < 8; ++w) { if (w < warp) woff += wsum[w]; tot += wsum[w]; }
    if (i < tiles) hd[i] = carry + woff + inc - v;
    carry += tot;
  }
}

// Stable scatter of one tile.  Elements are first ranked (warp by warp, in position order, so
// equal digits keep their order), then the tile is reordered by digit in shared memory so that
// the global writes are runs of consecutive addresses per digit.
template <bool FIRST, bool WITH_IDX>
__global__ void __launch_bounds__(TPB) long_scatter_kernel(const float* theta, const uint32_t* keys_in,
                                                           const int32_t* idx_in, uint32_t* keys_out,
                                                           int32_t* idx_out, const uint32_t* hist, int n,
                                                           int tiles, int shift, int mag) {
  __shared__ uint32_t cnt[WARPS][RADIX];     // running per-warp digit counts, then warp offsets inside the digit
  __shared__ uint32_t tstart[RADIX];         // first tile-local position of every digit
  __shared__ uint32_t gbase[RADIX];          // first global position of this tile's run of every digit
  __shared__ uint32_t skey[TILE];
  __shared__ int32_t sidx[WITH_IDX ? TILE : 1];   // indices travel only when a permutation is wanted
  const int tile = blockIdx.x;
  const long long row = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < WARPS * RADIX; i += TPB) (&cnt[0][0])[i] = 0;
  __syncthreads();
  const long long base = row * (long long)n;
  const int wstart = tile * TILE + warp * WCHUNK;
  uint32_t key[IPT];
  uint32_t lrank[IPT];                        // rank among the warp's earlier elements of the same digit
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int pos = wstart + i * 32 + lane;
    const bool valid = pos < n;
    uint32_t kk = 0xFFFFFFFFu;
    if (valid) kk = FIRST ? radix_key(__ldg(theta + base + pos), mag != 0) : keys_in[base + pos];
    key[i] = kk;
    const uint32_t digit = (kk >> shift) & 0xFF;
    // lanes with the same digit (invalid lanes form their own class and are ignored)
    const unsigned peers = __match_any_sync(0xffffffffu, valid ? digit : 0x100u);
    const unsigned lt = (1u << lane) - 1u;
    const int leader = __ffs(peers) - 1;
    uint32_t before = 0;
    if (valid && lane == leader) { before = cnt[warp][digit]; cnt[warp][digit] = before + __popc(peers); }
    before = __shfl_sync(0xffffffffu, before, leader);
    lrank[i] = before + __popc(peers & lt);
    __syncwarp();
  }
  __syncthreads();
  // per digit: offsets of the warps inside the digit, the digit's size in this tile, its global base
  for (int d = threadIdx.x; d < RADIX; d += TPB) {
    uint32_t run = 0;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) { uint32_t v = cnt[w][d]; cnt[w][d] = run; run += v; }
    tstart[d] = run;
    gbase[d] = hist[(row * RADIX + d) * (long long)tiles + tile];
  }
  __syncthreads();
  if (warp == 0) {      // exclusive scan of the 256 digit sizes, 8 per lane
    uint32_t v[8], sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[i] = tstart[lane * 8 + i]; sum += v[i]; }
    uint32_t inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
    uint32_t run = inc - sum;
#pragma unroll
    for (int i = 0; i < 8; ++i) { tstart[lane * 8 + i] = run; run += v[i]; }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int pos = wstart + i * 32 + lane;
    if (pos < n) {
      const uint32_t digit = (key[i] >> shift) & 0xFF;
      const uint32_t lp = tstart[digit] + cnt[warp][digit] + lrank[i];
      skey[lp] = key[i];
      if (WITH_IDX) sidx[lp] = FIRST ? pos : idx_in[base + pos];
    }
  }
  __syncthreads();
  const int count = min(TILE, n - tile * TILE);
  for (int j = threadIdx.x; j < count; j += TPB) {
    const uint32_t kk = skey[j];
    const uint32_t digit = (kk >> shift) & 0xFF;
    const uint32_t dst = gbase[digit] + ((uint32_t)j - tstart[digit]);
    keys_out[base + dst] = kk;
    if (WITH_IDX) idx_out[base + dst] = sidx[j];
  }
}

__global__ void long_export_sort_kernel(const uint32_t* keys, const int32_t* idx, int32_t* perm_out,
                                        float* sorted_out, long long total) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  if (perm_out) perm_out[i] = idx[i];
  if (sorted_out) sorted_out[i] = radix_key_to_float(keys[i]);
}

// ---- solve ---------------------------------------------------------------------
struct RowSetup { float c, vtop_c, piv, W_hi, W_lo; bool has_block; };

__device__ __forceinline__ RowSetup row_setup(const Math& M, const uint32_t* skeys, int n, int k) {
  RowSetup s;
  s.c = radix_key_to_float(skeys[k - 1]);
  s.vtop_c = M.vtop(s.c);
  s.has_block = (k < n) && (s.vtop_c < radix_key_to_float(skeys[k]));
  s.piv = (M.mag && s.vtop_c < 0.5f * s.c) ? 0.0f : s.c;
  s.W_hi = (s.piv == s.c) ? M.width(s.c) : s.c + M.width(s.c);
  s.W_lo = s.vtop_c - s.piv;
  return s;
}

// in-tile exclusive prefix sums of d^m over the window + tile totals
__global__ void __launch_bounds__(TPB) long_prefix_kernel(const Problem P, LongWs ws, int tiles) {
  __shared__ float wtot[3][WARPS];
  const int tile = blockIdx.x;
  const long long row = blockIdx.y;
  const int n = P.n, k = P.k;
  const Math M = make_math_q24(P);
  const uint32_t* skeys = ws.keyB + row * (long long)n;
  const RowSetup S = row_setup(M, skeys, n, k);
  if (!S.has_block) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  {
    // A tile with no rank inside the window has nothing to sum: all of it capped (its last key at or
    // above the window), or all of it below (its first key at or below the window).  The search only
    // reads prefix sums at ranks wl..wh; of a skipped tile that can only be its first rank (= wh).
    const int first = tile * TILE, last = min(first + TILE, n) - 1;
    const float d_first = radix_key_to_float(skeys[first]) - S.piv;
    const float d_last = radix_key_to_float(skeys[last]) - S.piv;
    if (d_last >= S.W_hi || !(d_first > S.W_lo)) {
      if (threadIdx.x == 0) {
        const long long base0 = row * (long long)n;
        ws.pin1[base0 + first] = 0.0f;
        if (M.q4) { ws.pin2[base0 + first] = 0.0f; ws.pin3[base0 + first] = 0.0f; }
        double* ts = ws.tsum + row * 3ll * tiles;
        ts[tile] = 0.0; ts[tiles + tile] = 0.0; ts[2 * tiles + tile] = 0.0;
      }
      return;
    }
  }
  const int start = tile * TILE + threadIdx.x * IPT;     // blocked: 16 consecutive ranks per thread
  float e1[IPT], e2[IPT], e3[IPT];
  float s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int pos = start + i;
    e1[i] = s1; e2[i] = s2; e3[i] = s3;
    if (pos < n) {
      const float d = radix_key_to_float(skeys[pos]) - S.piv;
      if (d > S.W_lo && !(d >= S.W_hi)) { s1 += d; const float d2 = d * d; s2 += d2; s3 += d2 * d; }
    }
  }
  // block exclusive scan of (s1, s2, s3)
  float i1 = s1, i2 = s2, i3 = s3;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    float u1 = __shfl_up_sync(0xffffffffu, i1, o), u2 = __shfl_up_sync(0xffffffffu, i2, o),
          u3 = __shfl_up_sync(0xffffffffu, i3, o);
    if (lane >= o) { i1 += u1; i2 += u2; i3 += u3; }
  }
  if (lane == 31) { wtot[0][warp] = i1; wtot[1][warp] = i2; wtot[2][warp] = i3; }
  __syncthreads();
  float o1 = i1 - s1, o2 = i2 - s2, o3 = i3 - s3;
  float t1 = 0.f, t2 = 0.f, t3 = 0.f;
  for (int w = 0; w < WARPS; ++w) {
    if (w < warp) { o1 += wtot[0][w]; o2 += wtot[1][w]; o3 += wtot[2][w]; }
    t1 += wtot[0][w]; t2 += wtot[1][w]; t3 += wtot[2][w];
  }
  const long long base = row * (long long)n;
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int pos = start + i;
    if (pos < n) {
      ws.pin1[base + pos] = o1 + e1[i];
      if (M.q4) { ws.pin2[base + pos] = o2 + e2[i]; ws.pin3[base + pos] = o3 + e3[i]; }
    }
  }
  if (threadIdx.x == 0) {
    double* ts = ws.tsum + row * 3ll * tiles;
    ts[tile] = (double)t1; ts[tiles + tile] = (double)t2; ts[2 * tiles + tile] = (double)t3;
  }
}

template <typename T>
__device__ __forceinline__ T block_sum_1024(T v, T* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  T w = (lane < nw) ? red[lane] : T(0);
  w = warp_sum(w);
  __syncthreads();
  return w;
}

// one block per row: tile offsets, window bounds, search of [a, b), block value
__global__ void __launch_bounds__(1024) long_solve_kernel(const Problem P, LongWs ws, int tiles,
                                                          tk_rowstate* state) {
  __shared__ double redd[32];
  __shared__ int sh_lo, sh_hi;
  __shared__ float sh_u;
  const long long row = blockIdx.x;
  const int n = P.n, k = P.k, t = threadIdx.x, T = blockDim.x;
  const Math M = make_math_q24(P);
  const bool mag = M.mag;
  const uint32_t* skeys = ws.keyB + row * (long long)n;
  const RowSetup S = row_setup(M, skeys, n, k);
  auto sval = [&](int i) -> float { return radix_key_to_float(skeys[i]); };
  int a0 = k, b0 = k;
  float u = 0.0f;
  if (S.has_block) {        // uniform over the block
    double* ts = ws.tsum + row * 3ll * tiles;
    // exclusive scan of the tile totals: warps 0..2 take one moment each, 32 tiles at a time
    if (t < 96) {
      const int lane = t & 31;
      double* a = ts + (long long)(t >> 5) * tiles;
      double carry = 0.0;
      for (int i0 = 0; i0 < tiles; i0 += 32) {
        const int i = i0 + lane;
        const double v = (i < tiles) ? a[i] : 0.0;
        double inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { double up = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += up; }
        if (i < tiles) a[i] = carry + inc - v;
        carry += __shfl_sync(0xffffffffu, inc, 31);
      }
    }
    __syncthreads();
    const float* pin1 = ws.pin1 + row * (long long)n;
    const float* pin2 = ws.pin2 + row * (long long)n;
    const float* pin3 = ws.pin3 + row * (long long)n;
    const float piv = S.piv;
    auto count_ge = [&](float x, int L, int R) -> int {
      while (L < R) { int mid = (L + R) >> 1; if (sval(mid) - piv >= x) L = mid + 1; else R = mid; }
      return L;
    };
    auto count_gt = [&](float x, int L, int R) -> int {
      while (L < R) { int mid = (L + R) >> 1; if (sval(mid) - piv > x) L = mid + 1; else R = mid; }
      return L;
    };
    const int wl = count_ge(S.W_hi, 0, k);
    const int wh = count_gt(S.W_lo, k, n);
    // prefix of d^m over window ranks below r (r <= n)
    auto prefix = [&](int r, double& q1, double& q2, double& q3) {
      if (r >= n) {       // total: last tile's offset + its in-tile total, recomputed from the last element
        const int last = n - 1, tl = last / TILE;
        const float d = sval(last) - piv;
        const bool in = d > S.W_lo && !(d >= S.W_hi);
        q1 = ts[tl] + (double)pin1[last] + (in ? (double)d : 0.0);
        q2 = q3 = 0.0;
        if (M.q4) {
          q2 = ts[tiles + tl] + (double)pin2[last] + (in ? (double)d * d : 0.0);
          q3 = ts[2 * tiles + tl] + (double)pin3[last] + (in ? (double)d * d * d : 0.0);
        }
        return;
      }
      const int tl = r / TILE;
      q1 = ts[tl] + (double)pin1[r];
      q2 = q3 = 0.0;
      if (M.q4) { q2 = ts[tiles + tl] + (double)pin2[r]; q3 = ts[2 * tiles + tl] + (double)pin3[r]; }
    };
    auto evalF = [&](float uu, int r_hi, int r_lo) -> float {
      double h1, h2, h3, l1, l2, l3;
      prefix(r_hi, h1, h2, h3);
      prefix(r_lo, l1, l2, l3);
      const float cnt = (float)(r_lo - r_hi);
      const float D1 = (float)(l1 - h1);
      float Sx;
      if (M.q4) {
        const float D2 = (float)(l2 - h2), D3 = (float)(l3 - h3);
        Sx = (((-cnt * uu + 3.0f * D1) * uu - 3.0f * D2) * uu + D3) * (P.inv_lam * P.inv_lam * P.inv_lam);
      } else {
        Sx = (D1 - cnt * uu) * P.inv_lam;
      }
      if (mag) Sx = Sx / (piv + uu);
      return (float)(r_hi - k) + Sx;
    };
    auto predB = [&](int j) -> bool {
      if (j < k) return true;
      if (j >= wh) return false;
      const float tau = sval(j);
      const float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      const int r_hi = count_ge(uu + M.width(tau), wl, k);
      return evalF(uu, r_hi, j) < 0.0f;
    };
    auto predA = [&](int j) -> bool {
      if (j < wl) return true;
      if (j >= k) return false;
      const float tau = M.vtop(sval(j));
      const float uu = tau - piv;
      if (mag && !(tau > 0.0f)) return false;
      const int r_lo = count_gt(uu, k, wh);
      return evalF(uu, j, r_lo) <= 0.0f;
    };
    // T-ary search: b0 = number of ranks with predB true in [k, wh]; bounded rounds
    int lo = k, hi = wh;            // predB(lo - 1) true (or lo == k), predB(hi) false
    for (int round = 0; round < 8 && hi - lo > 0; ++round) {
      const int span = hi - lo;
      const int step = (span + T - 1) / T;
      const int j = lo + t * step;                       // probes lo, lo+step, ...
      const bool pr = (j < hi) ? predB(j) : false;
      const int cntp = __syncthreads_count(pr);          // probes are monotone: true prefix
      if (t == 0) {
        // boundary in (lo + (cntp-1)*step, lo + cntp*step]
        sh_lo = (cntp == 0) ? lo : min(lo + (cntp - 1) * step + 1, hi);
        sh_hi = (cntp == 0) ? lo : min(lo + cntp * step, hi);
      }
      __syncthreads();
      lo = sh_lo; hi = sh_hi;
      __syncthreads();
    }
    b0 = lo;
    lo = wl; hi = k;
    for (int round = 0; round < 8 && hi - lo > 0; ++round) {
      const int span = hi - lo;
      const int step = (span + T - 1) / T;
      const int j = lo + t * step;
      const bool pr = (j < hi) ? predA(j) : false;
      const int cntp = __syncthreads_count(pr);
      if (t == 0) {
        sh_lo = (cntp == 0) ? lo : min(lo + (cntp - 1) * step + 1, hi);
        sh_hi = (cntp == 0) ? lo : min(lo + cntp * step, hi);
      }
      __syncthreads();
      lo = sh_lo; hi = sh_hi;
      __syncthreads();
    }
    a0 = lo;
    b0 = min(max(b0, k + 1), wh);
    a0 = max(min(a0, k - 1), wl);
    // block sums over [a0, b0), directly, in double
    double f1 = 0.0, f2 = 0.0, f3 = 0.0;
    for (int i = a0 + t; i < b0; i += T) {
      const double d = (double)(sval(i) - piv);
      f1 += d; f2 += d * d; f3 += d * d * d;
    }
    const double D1 = block_sum_1024<double>(f1, redd);
    const double D2 = block_sum_1024<double>(f2, redd);
    const double D3 = block_sum_1024<double>(f3, redd);
    if (t == 0) {
      const double cnt = (double)(b0 - a0), m = (double)(k - a0);
      const double u_left = mag ? (double)S.W_lo : D1 / cnt - (double)P.lam * cbrt(m / cnt);
      int nc = 0;
      sh_u = (float)solve_block_u(M.q4, mag, (double)P.lam, (double)piv, cnt, m, D1, D2, D3, u_left, &nc);
      sh_u = settle_offset(M, piv, sh_u, a0, b0, n, sval);
      if (nc && P.status) atomicOr(P.status, TK_FLAG_NOT_CONVERGED);
    }
    __syncthreads();
    u = sh_u;
  }
  if (t == 0) {
    tk_rowstate st;
    st.pivot = S.has_block ? S.piv : S.c; st.offset = u; st.a = a0; st.b = b0;
    state[row] = st;
  }
}

// y in sorted coordinates, scattered to the original positions
__global__ void __launch_bounds__(256) long_map_kernel(const Problem P, LongWs ws, const tk_rowstate* state) {
  const long long row = blockIdx.y;
  const int n = P.n;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const Math M = make_math_q24(P);
  const tk_rowstate st = state[row];
  const bool has_block = st.b > st.a;
  const long long base = row * (long long)n;
  const float s = radix_key_to_float(ws.keyB[base + i]);
  const int idx = ws.idxB[base + i];
  float y;
  if (i < st.a) y = M.mag ? M.vtop(s) : 1.0f;
  else if (i < st.b) {
    const float wid = has_block ? M.width(st.pivot + st.offset) : 0.0f;
    y = M.rho(fminf(fmaxf((s - st.pivot) - st.offset, 0.0f), wid));
  } else y = 0.0f;
  if (P.mode != TK_MASK) {
    const float x = __ldg(P.theta + base + idx);
    if (M.mag) y = signbit(x) ? -y : y;
    else y *= x;
  }
  P.out[base + idx] = y;
}

// y placed by value, in the original order: the class of an element follows from its key, gamma
// and the block's width, so neither the permutation nor a scatter is needed.
__global__ void __launch_bounds__(256) long_map_value_kernel(const Problem P, const tk_rowstate* state) {
  const long long row = blockIdx.y;
  const int n = P.n;
  const Math M = make_math_q24(P);
  const tk_rowstate st = state[row];
  const bool has_block = st.b > st.a;
  const float wid = has_block ? M.width(st.pivot + st.offset) : 0.0f;
  const long long base = row * (long long)n;
  const int start = blockIdx.x * kLongTile;
#pragma unroll 4
  for (int j = 0; j < kLongTile / 256; ++j) {
    const int i = start + j * 256 + threadIdx.x;
    if (i < n) {
      const float x = __ldg(P.theta + base + i);
      const float key = sort_key(x, M.mag);
      const float d = key - st.pivot;
      int cls; float tt = 0.0f;
      if (!has_block) cls = d >= 0.0f ? 2 : 0;
      else { const float t = d - st.offset; tt = fminf(fmaxf(t, 0.0f), wid); cls = t >= wid ? 2 : (t > 0.0f ? 1 : 0); }
      float y = cls == 2 ? (M.mag ? M.vtop(key) : 1.0f) : (cls == 1 ? M.rho(tt) : 0.0f);
      if (M.mag) y = signbit(x) ? -y : y;
      if (P.mode == TK_TOPK) y *= x;
      P.out[base + i] = y;
    }
  }
}

LongWs carve(void* workspace, long long rows, int n, int tiles, size_t* total) {
  LongWs w{};
  size_t off = 0;
  const size_t el = (size_t)rows * (size_t)n;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  char* b = static_cast<char*>(workspace);
  size_t o;
  o = take(el * 4); w.keyA = reinterpret_cast<uint32_t*>(b + o);
  o = take(el * 4); w.keyB = reinterpret_cast<uint32_t*>(b + o);
  o = take(el * 4); w.idxA = reinterpret_cast<int32_t*>(b + o);
  o = take(el * 4); w.idxB = reinterpret_cast<int32_t*>(b + o);
  o = take((size_t)rows * RADIX * tiles * 4); w.hist = reinterpret_cast<uint32_t*>(b + o);
  o = take((size_t)rows * RADIX * 4); w.dtot = reinterpret_cast<uint32_t*>(b + o);
  o = take(el * 4); w.pin1 = reinterpret_cast<float*>(b + o);
  o = take(el * 4); w.pin2 = reinterpret_cast<float*>(b + o);
  o = take(el * 4); w.pin3 = reinterpret_cast<float*>(b + o);
  o = take((size_t)rows * 3 * tiles * 8); w.tsum = reinterpret_cast<double*>(b + o);
  o = take((size_t)rows * sizeof(tk_rowstate)); w.state = reinterpret_cast<tk_rowstate*>(b + o);
  *total = off;
  return w;
}

}  // namespace

size_t long_workspace_bytes(long long rows, int n) {
  size_t total = 0;
  const int tiles = (n + TILE - 1) / TILE;
  carve(nullptr, rows, n, tiles, &total);
  return total;
}

// Sorts every row; the result is in ws.keyB (and ws.idxB when the indices travel too).
static cudaError_t long_sort(const Problem& P, const LongWs& ws, int tiles, bool with_idx, cudaStream_t stream) {
  const dim3 grid((unsigned)tiles, (unsigned)P.rows);
  const int mag = P.mode == TK_TOPKMAG;
  const uint32_t* kin = nullptr; const int32_t* iin = nullptr;
  uint32_t* kout = ws.keyA; int32_t* iout = ws.idxA;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 8 * pass;
    if (pass == 0) long_hist_kernel<true><<<grid, TPB, 0, stream>>>(P.theta, nullptr, ws.hist, P.n, tiles, shift, mag, P.status);
    else long_hist_kernel<false><<<grid, TPB, 0, stream>>>(nullptr, kin, ws.hist, P.n, tiles, shift, mag, nullptr);
    if (tiles > 64) {
      const dim3 dgrid(RADIX, (unsigned)P.rows);
      long_digit_total_kernel<<<dgrid, 256, 0, stream>>>(ws.hist, ws.dtot, tiles);
      long_digit_scan_kernel<<<dgrid, 256, 0, stream>>>(ws.hist, ws.dtot, tiles);
    } else {
      long_scan_hist_kernel<<<(unsigned)P.rows, 1024, 0, stream>>>(ws.hist, tiles);
    }
    if (pass == 0) {
      if (with_idx) long_scatter_kernel<true, true><<<grid, TPB, 0, stream>>>(P.theta, nullptr, nullptr, kout, iout, ws.hist, P.n, tiles, shift, mag);
      else long_scatter_kernel<true, false><<<grid, TPB, 0, stream>>>(P.theta, nullptr, nullptr, kout, iout, ws.hist, P.n, tiles, shift, mag);
    } else {
      if (with_idx) long_scatter_kernel<false, true><<<grid, TPB, 0, stream>>>(nullptr, kin, iin, kout, iout, ws.hist, P.n, tiles, shift, mag);
      else long_scatter_kernel<false, false><<<grid, TPB, 0, stream>>>(nullptr, kin, iin, kout, iout, ws.hist, P.n, tiles, shift, mag);
    }
    kin = kout; iin = iout;
    if (kout == ws.keyA) { kout = ws.keyB; iout = ws.idxB; } else { kout = ws.keyA; iout = ws.idxA; }
  }
  return cudaGetLastError();    // four passes: A, B, A, B -> result in B
}

// Forward pass, argsort, or (skip_map) only the row state, for rows of any length.
cudaError_t launch_long(const Problem& P, void* workspace, tk_rowstate* state_dst, bool skip_map,
                        cudaStream_t stream) {
  const int tiles = (P.n + TILE - 1) / TILE;
  size_t total = 0;
  LongWs ws = carve(workspace, P.rows, P.n, tiles, &total);
  // the indices ride along only when the caller asks for the permutation
  const bool with_idx = P.perm_out != nullptr || P.what == W_ARGSORT;
  cudaError_t e = long_sort(P, ws, tiles, with_idx, stream);
  if (e != cudaSuccess) return e;
  const long long el = P.rows * (long long)P.n;
  if (P.perm_out || P.sorted_out)
    long_export_sort_kernel<<<(unsigned)((el + 255) / 256), 256, 0, stream>>>(ws.keyB, ws.idxB, P.perm_out,
                                                                              P.sorted_out, el);
  if (P.what == W_ARGSORT) return cudaGetLastError();
  tk_rowstate* state = state_dst ? state_dst : ws.state;
  const dim3 grid((unsigned)tiles, (unsigned)P.rows);
  long_prefix_kernel<<<grid, TPB, 0, stream>>>(P, ws, tiles);
  long_solve_kernel<<<(unsigned)P.rows, 1024, 0, stream>>>(P, ws, tiles, state);
  if (!skip_map) {
    if (with_idx) {
      const dim3 mgrid((unsigned)((P.n + 255) / 256), (unsigned)P.rows);
      long_map_kernel<<<mgrid, 256, 0, stream>>>(P, ws, state);      // un-permute: out[sigma_i] = y_i
    } else {
      long_map_value_kernel<<<grid, 256, 0, stream>>>(P, state);
    }
  }
  return cudaGetLastError();
}

// Where launch_long leaves the sorted rows: keys as the complemented order-preserving words (so that
// key2f(~word) is the key), idx the original index of each rank (W_ARGSORT or perm_out only).
void long_workspace_sorted(void* workspace, long long rows, int n, const uint32_t** keys, const int32_t** idx) {
  const int tiles = (n + TILE - 1) / TILE;
  size_t total = 0;
  const LongWs ws = carve(workspace, rows, n, tiles, &total);
  *keys = ws.keyB;
  *idx = ws.idxB;
}

tk_rowstate* long_workspace_state(void* workspace, long long rows, int n) {
  const int tiles = (n + TILE - 1) / TILE;
  size_t total = 0;
  return carve(workspace, rows, n, tiles, &total).state;
}

// rows * tiles * 16 bytes of scratch for the VJP's per-tile partial sums (the 24 bytes per tile of
// the solve's tile totals, dead by then)
void* long_workspace_partials(void* workspace, long long rows, int n) {
  const int tiles = (n + TILE - 1) / TILE;
  size_t total = 0;
  return carve(workspace, rows, n, tiles, &total).tsum;
}

}  // namespace tk
