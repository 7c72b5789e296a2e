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
// How: the scratch is a file-scope __device__ array.  It belongs to the library's
// module: a GPU carries TK_NOALLOC_SCRATCH_BYTES of it from the moment the CUDA
// runtime loads that module on it (with lazy loading: this file's first lookup or
// launch on that GPU) until the process exits or resets the device.  In host code
// the array's name only stands for the symbol; its device address is looked up
// with cudaGetSymbolAddress, once per device, on the first call made with that
// device current -- which is therefore the call that can still fail for lack of
// memory, and the one to make at start-up.
#include <atomic>

#include "tk_common.cuh"

namespace tk {
size_t long_workspace_bytes(long long rows, int n);
cudaError_t launch_long(const Problem& P, void* workspace, tk_rowstate* state_dst, bool skip_map,
                        cudaStream_t stream);
// the argument checks of the regular entry points, and the longest row they serve without scratch (tk_api.cu)
tk_status check_common(const void* theta, int64_t rows, int64_t n, int64_t k, double p, double lambda,
                       int mode, int* q4, double* qm1);
int max_key_only_n();
}  // namespace tk

namespace {

constexpr size_t kScratchBytes = TK_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
// Device address of g_scratch, per device ordinal.  Host threads that make the first call on a
// device at the same time each look the address up and store the same value: the atomic makes
// that store and the later loads well defined.  The address is that of the module instance loaded
// when it was looked up: after cudaDeviceReset it is stale and this entry point must not be used.
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Device address of the scratch array on the current device (looked up once).
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    e = cudaGetSymbolAddress(&p, g_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return cudaSuccess;
}

}  // namespace

extern "C" tk_status tk_fwd_noalloc(const float* theta, int64_t rows, int64_t n, int64_t k, double p,
                                    double lambda, int mode, float* out, tk_stream stream) {
  // shapes that need no scratch go through the regular entry point unchanged
  if (n <= tk::max_key_only_n()) return tk_fwd(theta, rows, n, k, p, lambda, mode, out, stream);
  // the argument checks of tk_fwd_ex, before anything touches the device
  int q4 = 0;
  double qm1 = 0.0;
  const tk_status cs = tk::check_common(theta, rows, n, k, p, lambda, mode, &q4, &qm1);
  if (cs != TK_OK) return cs;
  if (qm1 > 0.0) return TK_ERR_UNSUPPORTED;
  if (rows == 0) return TK_OK;
  if (out == nullptr) return TK_ERR_INVALID_ARG;
  if (rows > 65535) return TK_ERR_UNSUPPORTED;
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
