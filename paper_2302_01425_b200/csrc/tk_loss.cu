// tk_loss.cu -- the smooth top-k loss of Sec. 6 ("Smooth top-k loss"):
//   loss(x, t) = f(x, 1_k) - <x, t>,   f(x, 1_k) = max_{y in P(1_k)} <y, x> - R(y),
// with phi(x) = x (Prop. "Relaxed operator": the maximiser is the relaxed top-k
// mask y*, and grad_1 f = y*), R(y) = (lambda/p) sum y_i^p, t one-hot.
//
// The forward pass has already written y* into `grad`; this pass reads x and y*
// once, reduces  sum_i y_i (x_i - (lambda/p) y_i^(p-1))  per row (most y_i are
// exactly 0 or 1), subtracts x[target] and turns y* into the gradient y* - t.
#include "tk_common.cuh"

namespace tk {

namespace {

enum { PK_2 = 0, PK_43 = 1, PK_GEN = 2 };

template <int PK>
__device__ __forceinline__ double loss_term(float x, float y, float lam_over_p, float pm1) {
  if (!(y > 0.0f)) return 0.0;
  const float ypm1 = (PK == PK_2) ? y : (PK == PK_43 ? cbrtf(y) : powf(y, pm1));
  return (double)y * ((double)x - (double)(lam_over_p * ypm1));
}

template <int PK, int TPR>      // TPR threads share a row: 32 (a warp) or 256 (the block)
__global__ void __launch_bounds__(256) tk_loss_kernel(const float* __restrict__ theta,
                                                      const int32_t* __restrict__ target, float* grad,
                                                      float* __restrict__ loss, long long rows, int n,
                                                      float lam_over_p, float pm1, int vec4) {
  constexpr int RPB = 256 / TPR;
  __shared__ double part[8];
  const int lane = threadIdx.x % TPR;
  const long long row = (long long)blockIdx.x * RPB + threadIdx.x / TPR;
  const bool live = row < rows;
  double acc = 0.0;
  const float* x = theta + (live ? row : 0) * (long long)n;
  float* y = grad + (live ? row : 0) * (long long)n;
  if (live) {
    if (vec4) {
      const float4* x4 = reinterpret_cast<const float4*>(x);
      const float4* y4 = reinterpret_cast<const float4*>(y);
      for (int i = lane; i < n / 4; i += TPR) {
        const float4 a = __ldg(x4 + i), b = y4[i];
        acc += loss_term<PK>(a.x, b.x, lam_over_p, pm1) + loss_term<PK>(a.y, b.y, lam_over_p, pm1);
        acc += loss_term<PK>(a.z, b.z, lam_over_p, pm1) + loss_term<PK>(a.w, b.w, lam_over_p, pm1);
      }
    } else {
      for (int i = lane; i < n; i += TPR) acc += loss_term<PK>(__ldg(x + i), y[i], lam_over_p, pm1);
    }
  }
  acc = warp_sum(acc);
  if (TPR > 32) {
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    acc = 0.0;
    if (threadIdx.x == 0)
      for (int w = 0; w < TPR / 32; ++w) acc += part[w];
  }
  // every read of this row's y* is complete (the shuffles, or the barrier, order it before this)
  if (live && lane == 0) {
    const int t = target ? __ldg(target + row) : -1;
    if (t >= 0 && t < n) {
      acc -= (double)__ldg(x + t);
      y[t] = y[t] - 1.0f;
    }
    loss[row] = (float)acc;
  }
}

template <int PK>
cudaError_t launch_pk(const float* theta, const int32_t* target, float* grad, float* loss, long long rows, int n,
                      float lam_over_p, float pm1, int vec4, cudaStream_t stream) {
  if (n <= 2048) {
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    tk_loss_kernel<PK, 32><<<blocks, 256, 0, stream>>>(theta, target, grad, loss, rows, n, lam_over_p, pm1, vec4);
  } else {
    tk_loss_kernel<PK, 256><<<(unsigned)rows, 256, 0, stream>>>(theta, target, grad, loss, rows, n, lam_over_p, pm1, vec4);
  }
  return cudaGetLastError();
}

}  // namespace

// grad holds the relaxed mask of every row on entry, mask - t on return; loss[r] as above.
cudaError_t launch_loss(const float* theta, const int32_t* target, float* grad, float* loss, long long rows,
                        int n, double p, double lambda, int q4, double qm1, int vec4, cudaStream_t stream) {
  const float lam_over_p = (float)(lambda / p), pm1 = (float)(p - 1.0);
  if (qm1 > 0.0) return launch_pk<PK_GEN>(theta, target, grad, loss, rows, n, lam_over_p, pm1, vec4, stream);
  if (q4) return launch_pk<PK_43>(theta, target, grad, loss, rows, n, lam_over_p, pm1, vec4, stream);
  return launch_pk<PK_2>(theta, target, grad, loss, rows, n, lam_over_p, pm1, vec4, stream);
}

}  // namespace tk
