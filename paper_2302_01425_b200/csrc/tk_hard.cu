// tk_hard.cu -- the hard operators of Sec. 3 read off a row's sorting permutation: topkmask has
// ones at sigma_1..sigma_k, topk = x * topkmask(x), topkmag = x * topkmask(|x|).  Used by the
// straight-through option (Sec. 6: hard top-k in the forward pass, the relaxed operator's gradient
// in the backward pass), after the forward pass has produced the permutation and the row state.
#include "tk_common.cuh"

namespace tk {

namespace {

// perm[r, i] = original index of the i-th largest key of row r.  One thread per (row, rank); the
// stores of a row land inside that row (n * 4 bytes), which the forward pass has just written.
__global__ void __launch_bounds__(256) tk_hard_kernel(const float* __restrict__ theta,
                                                      const int32_t* __restrict__ perm, float* out,
                                                      long long total, int n, int k, int mode) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long row = e / n;
    const int rank = (int)(e - row * n);
    const long long dst = row * n + __ldg(perm + e);
    float v = 0.0f;
    if (rank < k) v = (mode == TK_MASK) ? 1.0f : __ldg(theta + dst);
    out[dst] = v;
  }
}

}  // namespace

cudaError_t launch_hard(const float* theta, const int32_t* perm, float* out, long long rows, int n, int k,
                        int mode, cudaStream_t stream) {
  const long long total = rows * (long long)n;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)sm_count() * 64;  // grid-stride beyond a few waves
  if (blocks > cap) blocks = cap;
  tk_hard_kernel<<<(unsigned)blocks, 256, 0, stream>>>(theta, perm, out, total, n, k, mode);
  return cudaGetLastError();
}

}  // namespace tk
