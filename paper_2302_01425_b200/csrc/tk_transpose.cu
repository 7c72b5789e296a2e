// tk_transpose.cu -- tiled transpose between a [n, cols] matrix with leading dimension ld (the
// operator runs along its slow axis: problem c is column c) and the contiguous [cols, n] layout
// of the row kernels.  32 x 32 tiles through shared memory: both the loads and the stores of a
// warp are 128 contiguous bytes.
#include "tk_common.cuh"

namespace tk {

namespace {

// out[c * out_ld + r] = in[r * in_ld + c] for r < in_rows, c < in_cols
__global__ void __launch_bounds__(256) tk_transpose_kernel(const float* __restrict__ in, long long in_rows,
                                                           long long in_cols, long long in_ld,
                                                           float* __restrict__ out, long long out_ld) {
  __shared__ float tile[32][33];
  // tiles are numbered along a 1-D grid (either side of the matrix can exceed the 65535 blocks of gridDim.y)
  const long long tiles_c = (in_cols + 31) / 32;
  const long long c0 = ((long long)blockIdx.x % tiles_c) * 32, r0 = ((long long)blockIdx.x / tiles_c) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;        // 32 x 8 threads
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const long long r = r0 + ty + j, c = c0 + tx;
    if (r < in_rows && c < in_cols) tile[ty + j][tx] = __ldg(in + r * in_ld + c);
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const long long c = c0 + ty + j, r = r0 + tx;
    if (r < in_rows && c < in_cols) out[c * out_ld + r] = tile[tx][ty + j];
  }
}

}  // namespace

cudaError_t launch_transpose(const float* in, long long in_rows, long long in_cols, long long in_ld, float* out,
                             long long out_ld, cudaStream_t stream) {
  const long long tiles = ((in_cols + 31) / 32) * ((in_rows + 31) / 32);
  if (tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
  tk_transpose_kernel<<<(unsigned)tiles, 256, 0, stream>>>(in, in_rows, in_cols, in_ld, out, out_ld);
  return cudaGetLastError();
}

}  // namespace tk
