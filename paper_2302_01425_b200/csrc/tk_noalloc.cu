// tk_noalloc.cu -- forward pass for long rows with the scratch memory built
// into the library instead of supplied by the caller.
//
// Who this is for: code that has device buffers for its inputs and outputs but
// cannot obtain more device memory at the time of the call -- a plugin running
// inside a host application that owns the allocator, a callback in a real-time
// loop where cudaMalloc's implicit synchronisation is not acceptable, or a
// process whose memory pool is already fully committed.  The regular entry
// points make such callers size and pass a workspace for rows longer than
// 16384 elements; this one does not.
//
// How: the scratch is a file-scope __device__ array.  It is part of the loaded
// module, so every GPU that loads the library carries TK_NOALLOC_SCRATCH_BYTES
// of it until the process exits, whether or not this entry point is ever used.
// In host code the array's name only stands for the symbol; its device address
// is looked up with cudaGetSymbolAddress, once per device, on the first call
// made with that device current.
#include "tk_common.cuh"

namespace tk {
size_t long_workspace_bytes(long long rows, int n);
cudaError_t launch_long(const Problem& P, void* workspace, tk_rowstate* state_dst, bool skip_map,
                        cudaStream_t stream);
}  // namespace tk

namespace {

constexpr size_t kScratchBytes = TK_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_scratch, per device ordinal

// Device address of the scratch array on the current device (looked up once).
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" tk_status tk_fwd_noalloc(const float* theta, int64_t rows, int64_t n, int64_t k, double p,
                                    double lambda, int mode, float* out, tk_stream stream) {
  // shapes that need no scratch go through the regular entry point unchanged
  if (n <= 16384) return tk_fwd(theta, rows, n, k, p, lambda, mode, out, stream);
  // the same argument checks as tk_fwd_ex, before anything touches the device
  if (rows < 0 || k < 1 || k > n) return TK_ERR_INVALID_ARG;
  if (mode < TK_MASK || mode > TK_TOPKMAG) return TK_ERR_INVALID_ARG;
  if (!(lambda > 0.0) || !isfinite(lambda)) return TK_ERR_INVALID_ARG;
  if (!(p > 1.0) || !isfinite(p)) return TK_ERR_INVALID_ARG;
  const double q = p / (p - 1.0);
  int q4;
  if (fabs(q - 2.0) <= 1e-6) q4 = 0;
  else if (fabs(q - 4.0) <= 1e-6) q4 = 1;
  else return TK_ERR_UNSUPPORTED;
  if (rows == 0) return TK_OK;
  if (theta == nullptr || out == nullptr) return TK_ERR_INVALID_ARG;
  if (rows > 65535 || n > 0x7fffffff) return TK_ERR_UNSUPPORTED;
  // the built-in scratch has a fixed size: larger problems are refused, never truncated
  if ((double)rows * (double)n > (double)TK_NOALLOC_MAX_ELEMENTS) return TK_ERR_WORKSPACE;
  if (tk::long_workspace_bytes(rows, (int)n) > kScratchBytes) return TK_ERR_WORKSPACE;

  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return TK_ERR_CUDA;

  tk::Problem P{};
  P.theta = theta;
  P.out = out;
  P.rows = rows; P.n = (int)n; P.k = (int)k; P.q4 = q4; P.mode = mode;
  P.lam = (float)lambda;
  P.inv_lam = (float)(1.0 / lambda);
  P.lam3 = (float)(lambda * lambda * lambda);
  P.what = tk::W_FWD;
  // Nothing in the scratch has to start at zero: every word a kernel of this pipeline reads
  // (sort buffers, histograms, prefix sums, tile totals, row state) is written earlier in the
  // same call, so the previous call's contents are simply overwritten.
  cudaError_t e = tk::launch_long(P, scratch, nullptr, false, (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}
