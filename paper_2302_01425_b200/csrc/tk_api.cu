// tk_api.cu -- the C ABI: argument checks and dispatch.  Declarations and the
// meaning of every argument are in include/tk.h.
#include <math.h>

#include "tk_common.cuh"

namespace tk {
// on-chip row kernels (tk_cta.cu)
cudaError_t launch_cta(const Problem& P, cudaStream_t stream);
int cta_padded_length(int n);
// sub-warp row kernels for n <= 512 with the permutation (tk_group.cu); key-only sort and results
// by value for rows of up to 1024 elements (tk_rows.cu)
cudaError_t launch_group(const Problem& P, cudaStream_t stream);
cudaError_t launch_rows(const Problem& P, cudaStream_t stream);
// block-per-row kernel with a key-only sort and results by value (tk_ctav.cu)
cudaError_t launch_ctav(const Problem& P, cudaStream_t stream);
// exact forward pass without a sort (tk_thr.cu); the same for phi(x) = x with rows in registers (tk_newton.cu)
cudaError_t launch_thr(const Problem& P, cudaStream_t stream);
cudaError_t launch_newton(const Problem& P, cudaStream_t stream);
int newton_max_n();
// the same for a few rows of any length, the row in global memory (tk_long_newton.cu)
size_t long_newton_scratch_bytes();
cudaError_t launch_long_newton(const Problem& P, void* scratch, cudaStream_t stream);
// alternating-projection solver path (tk_dykstra.cu)
cudaError_t launch_dykstra(const Problem& P, cudaStream_t stream);
int dykstra_cluster_max_n();
cudaError_t launch_dykstra_cluster(const Problem& P, const uint32_t* keys, const int32_t* idx,
                                   cudaStream_t stream);
// smooth top-k loss from the relaxed mask (tk_loss.cu)
cudaError_t launch_loss(const float* theta, const int32_t* target, float* grad, float* loss, long long rows,
                        int n, double p, double lambda, int q4, double qm1, int vec4, cudaStream_t stream);
// hard operators from the permutation (tk_hard.cu)
cudaError_t launch_hard(const float* theta, const int32_t* perm, float* out, long long rows, int n, int k,
                        int mode, cudaStream_t stream);
// [n, cols] with leading dimension <-> contiguous [cols, n] (tk_transpose.cu)
cudaError_t launch_transpose(const float* in, long long in_rows, long long in_cols, long long in_ld, float* out,
                             long long out_ld, cudaStream_t stream);
// relaxed operator over the permutahedron of any sorted w (tk_w.cu)
int w_max_n();
cudaError_t launch_w(const Problem& P, const float* w, long long w_rows, cudaStream_t stream);
// VJP from saved row state (tk_vjp_state.cu)
cudaError_t launch_vjp_state(const Problem& P, cudaStream_t stream);
cudaError_t launch_vjp_state_long(const Problem& P, void* scratch, cudaStream_t stream);
// rows held in global memory (tk_long.cu)
size_t long_workspace_bytes(long long rows, int n);
cudaError_t launch_long(const Problem& P, void* workspace, tk_rowstate* state_dst, bool skip_map,
                        cudaStream_t stream);
tk_rowstate* long_workspace_state(void* workspace, long long rows, int n);
void* long_workspace_partials(void* workspace, long long rows, int n);
void long_workspace_sorted(void* workspace, long long rows, int n, const uint32_t** keys, const int32_t** idx);

constexpr int kMaxOnChipN = 16384;   // longest row the block-per-row kernels hold in shared memory
constexpr int kMaxKeyOnlyN = 32768;  // longest row the key-only forward pass holds on chip (no workspace)
constexpr int kMaxGeneralSortedN = 128;   // general p: longest row solved by one lane's Newton iteration (tk_rows.cu)
constexpr int kMaxGroupN = 512;      // longest row a single warp holds in registers as (key, index) words
constexpr int kMaxWalkN = 1024;      // longest row of the warp-autonomous kernel (tk_rows.cu)

inline cudaError_t launch_on_chip(const Problem& P, cudaStream_t stream) {
  // Without a permutation to return, short rows sort their keys only and place results by value.
  const bool needs_perm = P.perm_out != nullptr || P.sorted_out != nullptr || P.what == W_ARGSORT;
  if (!needs_perm) {
    if (P.n <= kMaxWalkN) return launch_rows(P, stream);
    return launch_ctav(P, stream);
  }
  return P.n <= kMaxGroupN ? launch_group(P, stream) : launch_cta(P, stream);
}

// q = p/(p-1): 2 and 4 (p = 2, p = 4/3) have closed-form block solves and run everywhere.  Any
// other 1 < p < 2 (q > 2) is *qm1 = q - 1 > 0: forward pass by the sort-free solver, VJP from
// saved state for q >= 3.  Not supported: q < 2 (p > 2: rho' unbounded at 0); for 2 < q < 3
// (1.5 < p < 2) rho'' is unbounded at 0 and an fp32 key difference cannot carry the VJP of a barely
// pooled element to 1e-5, so only the forward pass (and the loss, whose gradient is the forward
// output) is served there (vjp_supported).
tk_status classify_p(double p, int* q4, double* qm1) {
  *q4 = 0; *qm1 = 0.0;
  if (!(p > 1.0) || !isfinite(p)) return TK_ERR_INVALID_ARG;
  double q = p / (p - 1.0);
  if (fabs(q - 2.0) <= 1e-6) return TK_OK;
  if (fabs(q - 4.0) <= 1e-6) { *q4 = 1; return TK_OK; }
  if (!(q > 2.0) || q > 64.0) return TK_ERR_UNSUPPORTED;
  *qm1 = q - 1.0;
  return TK_OK;
}

tk_status check_common(const void* theta, int64_t rows, int64_t n, int64_t k, double p,
                       double lambda, int mode, int* q4, double* qm1) {
  if (rows < 0 || n < 1 || k < 1 || k > n) return TK_ERR_INVALID_ARG;
  if (mode < TK_MASK || mode > TK_TOPKMAG) return TK_ERR_INVALID_ARG;
  if (!(lambda > 0.0) || !isfinite(lambda)) return TK_ERR_INVALID_ARG;
  tk_status s = classify_p(p, q4, qm1);
  if (s == TK_OK && *qm1 > 0.0 && n > kMaxOnChipN) s = TK_ERR_UNSUPPORTED;
  if (s != TK_OK) return s;
  if (rows > 0 && theta == nullptr) return TK_ERR_INVALID_ARG;
  if (n > 0x7fffffff || rows > 0x7fffffffLL) return TK_ERR_UNSUPPORTED;
  return TK_OK;
}

int max_key_only_n() { return kMaxKeyOnlyN; }
}  // namespace tk

namespace {

using tk::check_common;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Long rows need the caller's scratch: present, 256-byte aligned and large enough.
tk_status check_workspace(const tk_opts* opts, int64_t rows, int64_t n) {
  if (rows > 65535) return TK_ERR_UNSUPPORTED;            // rows ride on gridDim.y there
  if (!opts || !opts->workspace) return TK_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(opts->workspace) & 255u) return TK_ERR_WORKSPACE;
  if (opts->workspace_bytes < tk::long_workspace_bytes(rows, (int)n)) return TK_ERR_WORKSPACE;
  return TK_OK;
}

// derivatives are served for q = 2, 4 and any q >= 3
bool vjp_supported(double qm1) { return qm1 == 0.0 || qm1 >= 2.0 - 1e-9; }

void fill(tk::Problem& P, const float* theta, int64_t rows, int64_t n, int64_t k, int q4,
          double qm1, double lambda, int mode) {
  P = tk::Problem{};
  P.theta = theta;
  P.rows = rows; P.n = (int)n; P.k = (int)k; P.q4 = q4; P.qm1 = (float)qm1; P.mode = mode;
  P.lam = (float)lambda;
  P.inv_lam = (float)(1.0 / lambda);
  P.lam3 = (float)(lambda * lambda * lambda);
}

}  // namespace

extern "C" {

const char* tk_version(void) { return "tk 0.1 sm_100a"; }

const char* tk_status_string(int status) {
  switch (status) {
    case TK_OK: return "ok";
    case TK_ERR_INVALID_ARG: return "invalid argument";
    case TK_ERR_UNSUPPORTED: return "unsupported configuration";
    case TK_ERR_WORKSPACE: return "workspace missing or too small";
    case TK_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

size_t tk_workspace_bytes(int64_t rows, int64_t n, int64_t k, double p, int mode, int solver) {
  (void)k; (void)solver;
  if (rows <= 0 || n > 0x7fffffff) return 0;
  if (n <= tk::kMaxOnChipN) {
    // a general p: tk_vjp without saved state runs the forward pass again and keeps its row state here
    int q4 = 0;
    double qm1 = 0.0;
    if (tk::classify_p(p, &q4, &qm1) == TK_OK && qm1 > 0.0 && (n > tk::kMaxGeneralSortedN || mode == TK_TOPKMAG))
      return (((size_t)rows * sizeof(tk_rowstate)) + 255u) & ~(size_t)255u;
    return 0;
  }
  return tk::long_workspace_bytes(rows, (int)n);
}

static tk_status fwd_relaxed(const float* theta, int64_t rows, int64_t n, int64_t k, double p,
                             double lambda, int mode, float* out, const tk_opts* opts, tk_stream stream) {
  int q4 = 0;
  double qm1 = 0.0;
  tk_status s = check_common(theta, rows, n, k, p, lambda, mode, &q4, &qm1);
  if (s != TK_OK) return s;
  if (rows == 0) return TK_OK;
  if (out == nullptr) return TK_ERR_INVALID_ARG;
  int solver = opts ? opts->solver : TK_SOLVER_AUTO;
  if (solver < TK_SOLVER_AUTO || solver > TK_SOLVER_THRESHOLD) return TK_ERR_INVALID_ARG;
  if (qm1 > 0.0) {
    // general p: no closed-form block solve.  Rows of up to 128 elements: the sorting kernel with a
    // per-row Newton iteration on the threshold function; longer rows (and every explicit request
    // for it): the sort-free solver.  No permutation output either way.
    // (TK_SOLVER_DYKSTRA: the dual coordinate ascent of App. A.8 with a root-solving pair step)
    if (solver == TK_SOLVER_PAV) return TK_ERR_UNSUPPORTED;
    if (opts && opts->perm_out && solver != TK_SOLVER_DYKSTRA) return TK_ERR_UNSUPPORTED;
    if (solver != TK_SOLVER_DYKSTRA && (n > tk::kMaxGeneralSortedN || mode == TK_TOPKMAG)) solver = TK_SOLVER_THRESHOLD;
  }
  tk::Problem P;
  fill(P, theta, rows, n, k, q4, qm1, lambda, mode);
  P.out = out;
  P.what = tk::W_FWD;
  if (opts) { P.perm_out = opts->perm_out; P.state_out = opts->state_out; P.status = opts->status_out; }
  P.vec4 = (n % 4 == 0) && aligned16(theta) && aligned16(out);
  // phi(x) = x with a closed-form block solve, nothing but values asked for: the threshold form needs no
  // order at all (TK_SOLVER_PAV keeps the sort)
  // (very short rows sort faster than they iterate: AUTO keeps the sort up to 8 elements, up to 16 for p = 4/3)
  const bool by_threshold = (solver == TK_SOLVER_THRESHOLD || (solver == TK_SOLVER_AUTO && n > (q4 ? 16 : 8))) &&
                            qm1 == 0.0 && P.perm_out == nullptr && n <= tk::newton_max_n();
  if (by_threshold) {
    cudaError_t en = tk::launch_newton(P, (cudaStream_t)stream);
    return en == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  // A few very long rows (the pruning row): the same iteration with the row streamed from L2, all SMs on
  // one row at a time.  Many long rows keep the sorting pipeline, which works on all of them at once.
  if ((solver == TK_SOLVER_AUTO || solver == TK_SOLVER_THRESHOLD) && qm1 == 0.0 && P.perm_out == nullptr &&
      n > tk::newton_max_n() && rows <= 16) {
    s = check_workspace(opts, rows, n);
    if (s != TK_OK) return s;
    if (opts->workspace_bytes < tk::long_newton_scratch_bytes()) return TK_ERR_WORKSPACE;
    cudaError_t eln = tk::launch_long_newton(P, opts->workspace, (cudaStream_t)stream);
    return eln == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  if (solver == TK_SOLVER_THRESHOLD) {
    // no sort, hence no permutation to return; rows held on chip only
    if (n > tk::kMaxOnChipN || (opts && opts->perm_out)) return TK_ERR_UNSUPPORTED;
    cudaError_t et = tk::launch_thr(P, (cudaStream_t)stream);
    return et == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  if (solver == TK_SOLVER_DYKSTRA) {
    // Forward pass only: the iterate stays on chip; no row state (the iterate of a fixed number of
    // sweeps has no exact block structure to save); phi even with p = 4/3 has no closed-form pair step.
    if (n > tk::dykstra_cluster_max_n() || (opts && opts->state_out)) return TK_ERR_UNSUPPORTED;
    // phi even with p = 4/3 (no closed-form pair step: the root-solving one) on rows of one thread block only
    if (mode == TK_TOPKMAG && q4 && n > tk::kMaxOnChipN) return TK_ERR_UNSUPPORTED;
    P.sweeps = opts ? opts->sweeps : 0;
    P.tol = opts ? opts->tol : 0.0f;
    if (!(P.tol >= 0.0f) || !isfinite(P.tol)) return TK_ERR_INVALID_ARG;
    if (P.tol > 0.0f && n > tk::kMaxOnChipN) return TK_ERR_UNSUPPORTED;   // rows of one thread block only
    if (n > tk::kMaxOnChipN) {
      // rows shared by a thread-block cluster: sorted in global memory first (needs the workspace)
      s = check_workspace(opts, rows, n);
      if (s != TK_OK) return s;
      tk::Problem A = P;
      A.what = tk::W_ARGSORT; A.out = nullptr;
      cudaError_t ea = tk::launch_long(A, opts->workspace, nullptr, true, (cudaStream_t)stream);
      if (ea != cudaSuccess) return TK_ERR_CUDA;
      const uint32_t* keys = nullptr; const int32_t* idx = nullptr;
      tk::long_workspace_sorted(opts->workspace, rows, (int)n, &keys, &idx);
      ea = tk::launch_dykstra_cluster(P, keys, idx, (cudaStream_t)stream);
      return ea == cudaSuccess ? TK_OK : TK_ERR_CUDA;
    }
    cudaError_t ed = tk::launch_dykstra(P, (cudaStream_t)stream);
    return ed == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  // Without a permutation to return, rows of up to 32768 elements are sorted (keys only) on chip and
  // need no workspace; one that is passed is left untouched.
  const bool key_only_on_chip = n <= tk::kMaxKeyOnlyN && P.perm_out == nullptr;
  if (n > tk::kMaxOnChipN && !key_only_on_chip) {
    s = check_workspace(opts, rows, n);
    if (s != TK_OK) return s;
    cudaError_t el = tk::launch_long(P, opts->workspace, opts->state_out, false, (cudaStream_t)stream);
    return el == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  cudaError_t e = tk::launch_on_chip(P, (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_fwd_ex(const float* theta, int64_t rows, int64_t n, int64_t k, double p,
                    double lambda, int mode, float* out, const tk_opts* opts, tk_stream stream) {
  const bool st = opts && (opts->flags & TK_OPT_STRAIGHT_THROUGH);
  if (opts && (opts->flags & ~TK_OPT_STRAIGHT_THROUGH)) return TK_ERR_INVALID_ARG;
  if (st && rows > 0 && opts->perm_out == nullptr) return TK_ERR_INVALID_ARG;
  if (st && opts->solver == TK_SOLVER_THRESHOLD) return TK_ERR_UNSUPPORTED;
  tk_status s = fwd_relaxed(theta, rows, n, k, p, lambda, mode, out, opts, stream);
  if (s != TK_OK || !st || rows == 0) return s;
  // the relaxed pass has left the permutation (and the row state); the hard operator replaces its output
  cudaError_t e = tk::launch_hard(theta, opts->perm_out, out, rows, (int)n, (int)k, mode, (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_fwd(const float* theta, int64_t rows, int64_t n, int64_t k, double p, double lambda,
                 int mode, float* out, tk_stream stream) {
  return tk_fwd_ex(theta, rows, n, k, p, lambda, mode, out, nullptr, stream);
}

tk_status tk_vjp(const float* theta, const float* grad_out, int64_t rows, int64_t n, int64_t k,
                 double p, double lambda, int mode, float* grad_theta, const tk_opts* opts,
                 tk_stream stream) {
  int q4 = 0;
  double qm1 = 0.0;
  tk_status s = check_common(theta, rows, n, k, p, lambda, mode, &q4, &qm1);
  if (s != TK_OK) return s;
  if (rows == 0) return TK_OK;
  if (grad_out == nullptr || grad_theta == nullptr) return TK_ERR_INVALID_ARG;
  if (!vjp_supported(qm1)) return TK_ERR_UNSUPPORTED;
  // general p: from saved state, or recomputed by the sorting kernel for rows of up to 128 elements (phi = x);
  // otherwise the forward pass runs again here -- its output goes to grad_theta, which the VJP overwrites
  // afterwards, its row state to the caller's workspace
  const tk_rowstate* recomputed = nullptr;
  const bool room_for_state = opts && opts->workspace && !(reinterpret_cast<uintptr_t>(opts->workspace) & 255u) &&
                              opts->workspace_bytes >= (size_t)rows * sizeof(tk_rowstate);
  const bool must_recompute = qm1 > 0.0 && (n > tk::kMaxGeneralSortedN || mode == TK_TOPKMAG);
  // p = 2 and p = 4/3 on rows the threshold form serves: with room for the row state the forward pass that
  // needs no sort runs again; without it the sorting kernels recompute inside the VJP kernel
  const bool may_recompute = qm1 == 0.0 && n <= tk::newton_max_n() && room_for_state;
  if (!(opts && opts->state_out) && (must_recompute || may_recompute)) {
    if (!room_for_state) return TK_ERR_WORKSPACE;
    tk_opts f = {};
    f.solver = TK_SOLVER_AUTO;
    f.state_out = static_cast<tk_rowstate*>(opts->workspace);
    f.status_out = opts->status_out;
    s = tk_fwd_ex(theta, rows, n, k, p, lambda, mode, grad_theta, &f, stream);
    if (s != TK_OK) return s;
    recomputed = f.state_out;
  }
  tk::Problem P;
  fill(P, theta, rows, n, k, q4, qm1, lambda, mode);
  P.gout = grad_out;
  P.out = grad_theta;
  P.what = tk::W_VJP;
  if (opts) P.status = opts->status_out;
  P.vec4 = (n % 4 == 0) && aligned16(theta) && aligned16(grad_out) && aligned16(grad_theta);
  cudaError_t e;
  if (n > tk::kMaxOnChipN && n <= tk::kMaxKeyOnlyN && (recomputed || (opts && opts->state_out))) {
    // from row state (saved, or just recomputed) a row of this length needs no scratch
    P.state_in = recomputed ? recomputed : opts->state_out;
    e = tk::launch_vjp_state(P, (cudaStream_t)stream);
  } else if (n > tk::kMaxOnChipN) {
    s = check_workspace(opts, rows, n);
    if (s != TK_OK) return s;
    P.state_in = opts->state_out;
    if (!P.state_in) {      // no saved state: sort and solve again, keep only the row state
      tk::Problem F = P;
      F.what = tk::W_FWD; F.out = nullptr; F.gout = nullptr;
      e = tk::launch_long(F, opts->workspace, nullptr, true, (cudaStream_t)stream);
      if (e != cudaSuccess) return TK_ERR_CUDA;
      P.state_in = tk::long_workspace_state(opts->workspace, rows, (int)n);
    }
    e = tk::launch_vjp_state_long(P, tk::long_workspace_partials(opts->workspace, rows, (int)n),
                                  (cudaStream_t)stream);
  } else if (recomputed || (opts && opts->state_out)) {
    P.state_in = recomputed ? recomputed : opts->state_out;
    e = tk::launch_vjp_state(P, (cudaStream_t)stream);
  } else {
    e = tk::launch_on_chip(P, (cudaStream_t)stream);
  }
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_jvp(const float* theta, const float* tangent, int64_t rows, int64_t n, int64_t k,
                 double p, double lambda, int mode, float* out_tangent, const tk_opts* opts,
                 tk_stream stream) {
  int q4 = 0;
  double qm1 = 0.0;
  tk_status s = check_common(theta, rows, n, k, p, lambda, mode, &q4, &qm1);
  if (s != TK_OK) return s;
  if (rows == 0) return TK_OK;
  if (tangent == nullptr || out_tangent == nullptr) return TK_ERR_INVALID_ARG;
  if (!(opts && opts->state_out) || !vjp_supported(qm1)) return TK_ERR_UNSUPPORTED;   // from the forward pass's row state only
  tk::Problem P;
  fill(P, theta, rows, n, k, q4, qm1, lambda, mode);
  P.gout = tangent;
  P.out = out_tangent;
  P.what = tk::W_VJP;
  P.jvp = 1;
  P.state_in = opts->state_out;
  P.status = opts->status_out;
  P.vec4 = (n % 4 == 0) && aligned16(theta) && aligned16(tangent) && aligned16(out_tangent);
  cudaError_t e;
  if (n <= tk::kMaxKeyOnlyN) {
    e = tk::launch_vjp_state(P, (cudaStream_t)stream);
  } else {
    s = check_workspace(opts, rows, n);
    if (s != TK_OK) return s;
    e = tk::launch_vjp_state_long(P, tk::long_workspace_partials(opts->workspace, rows, (int)n),
                                  (cudaStream_t)stream);
  }
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_topk_loss(const float* theta, const int32_t* target, int64_t rows, int64_t n, int64_t k,
                       double p, double lambda, float* loss, float* grad, const tk_opts* opts,
                       tk_stream stream) {
  int q4 = 0;
  double qm1 = 0.0;
  tk_status s = check_common(theta, rows, n, k, p, lambda, TK_MASK, &q4, &qm1);
  if (s != TK_OK) return s;
  if (rows == 0) return TK_OK;
  if (loss == nullptr || grad == nullptr || (opts && opts->flags)) return TK_ERR_INVALID_ARG;
  // the relaxed mask y* into grad (every check of the forward pass applies), then one pass over (theta, y*)
  s = tk_fwd_ex(theta, rows, n, k, p, lambda, TK_MASK, grad, opts, stream);
  if (s != TK_OK) return s;
  const int vec4 = (n % 4 == 0) && aligned16(theta) && aligned16(grad);
  cudaError_t e = tk::launch_loss(theta, target, grad, loss, rows, (int)n, p, lambda, q4, qm1, vec4,
                                  (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

// ---- the operator along the slow axis: transpose into the workspace, row kernels, transpose back
static size_t cols_slab_bytes(int64_t n, int64_t cols) {
  return ((size_t)n * (size_t)cols * sizeof(float) + 255) & ~size_t(255);
}

size_t tk_cols_workspace_bytes(int64_t n, int64_t cols) {
  if (n < 1 || cols < 1 || n > tk::kMaxOnChipN || cols > (int64_t(1) << 21)) return 0;
  return 3 * cols_slab_bytes(n, cols);
}

static tk_status check_cols(int64_t n, int64_t cols, int64_t ld, const tk_opts* opts, float** slab) {
  if (cols < 0 || n < 1 || ld < cols) return TK_ERR_INVALID_ARG;
  if (n > tk::kMaxOnChipN || cols > (int64_t(1) << 21)) return TK_ERR_UNSUPPORTED;
  if (cols == 0) return TK_OK;
  if (!opts || !opts->workspace || (reinterpret_cast<uintptr_t>(opts->workspace) & 255u)) return TK_ERR_WORKSPACE;
  if (opts->workspace_bytes < tk_cols_workspace_bytes(n, cols)) return TK_ERR_WORKSPACE;
  const size_t slab_bytes = cols_slab_bytes(n, cols);
  for (int i = 0; i < 3; ++i) slab[i] = reinterpret_cast<float*>(static_cast<char*>(opts->workspace) + i * slab_bytes);
  return TK_OK;
}

tk_status tk_fwd_cols(const float* theta, int64_t n, int64_t cols, int64_t ld, int64_t k, double p,
                      double lambda, int mode, float* out, const tk_opts* opts, tk_stream stream) {
  float* slab[3] = {nullptr, nullptr, nullptr};
  tk_status s = check_cols(n, cols, ld, opts, slab);
  if (s != TK_OK) return s;
  int q4 = 0; double qm1 = 0.0;
  s = check_common(theta, cols, n, k, p, lambda, mode, &q4, &qm1);
  if (s != TK_OK) return s;
  if (cols == 0) return TK_OK;
  if (out == nullptr) return TK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (tk::launch_transpose(theta, n, cols, ld, slab[0], n, st) != cudaSuccess) return TK_ERR_CUDA;
  tk_opts inner = *opts;
  inner.workspace = nullptr; inner.workspace_bytes = 0;
  s = tk_fwd_ex(slab[0], cols, n, k, p, lambda, mode, slab[1], &inner, stream);
  if (s != TK_OK) return s;
  return tk::launch_transpose(slab[1], cols, n, n, out, ld, st) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_vjp_cols(const float* theta, const float* grad_out, int64_t n, int64_t cols, int64_t ld,
                      int64_t k, double p, double lambda, int mode, float* grad_theta,
                      const tk_opts* opts, tk_stream stream) {
  float* slab[3] = {nullptr, nullptr, nullptr};
  tk_status s = check_cols(n, cols, ld, opts, slab);
  if (s != TK_OK) return s;
  // theta == NULL: the transposed copy a forward call left in the workspace (needs its row state too)
  const bool reuse = theta == nullptr && opts && opts->state_out != nullptr;
  int q4 = 0; double qm1 = 0.0;
  s = check_common(reuse ? (const void*)slab : (const void*)theta, cols, n, k, p, lambda, mode, &q4, &qm1);
  if (s != TK_OK) return s;
  if (cols == 0) return TK_OK;
  if (grad_out == nullptr || grad_theta == nullptr) return TK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (!reuse && tk::launch_transpose(theta, n, cols, ld, slab[0], n, st) != cudaSuccess) return TK_ERR_CUDA;
  if (tk::launch_transpose(grad_out, n, cols, ld, slab[1], n, st) != cudaSuccess) return TK_ERR_CUDA;
  tk_opts inner = *opts;
  inner.workspace = nullptr; inner.workspace_bytes = 0;
  s = tk_vjp(slab[0], slab[1], cols, n, k, p, lambda, mode, slab[2], &inner, stream);
  if (s != TK_OK) return s;
  return tk::launch_transpose(slab[2], cols, n, n, grad_theta, ld, st) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

// ---- any sorted w: relaxed linear maximisation over the permutahedron P(w)
static tk_status run_w(const float* theta, const float* w, const float* grad_out, int64_t rows, int64_t n,
                       int64_t w_rows, double p, double lambda, float* out, float* grad_w, const tk_opts* opts,
                       tk_stream stream, int what) {
  int q4 = 0;
  double qm1 = 0.0;
  tk_status s = check_common(theta, rows, n, 1, p, lambda, TK_MASK, &q4, &qm1);
  if (s != TK_OK) return s;
  if (w_rows != 1 && w_rows != rows) return TK_ERR_INVALID_ARG;
  if (qm1 > 0.0 || n > tk::w_max_n() || (opts && (opts->flags || opts->perm_out))) return TK_ERR_UNSUPPORTED;
  if (rows == 0) return TK_OK;
  if (w == nullptr || out == nullptr || (what == tk::W_VJP && grad_out == nullptr)) return TK_ERR_INVALID_ARG;
  tk::Problem P;
  fill(P, theta, rows, n, 1, q4, 0.0, lambda, TK_MASK);
  P.out = out;
  P.gout = grad_out;
  P.sorted_out = grad_w;
  P.what = what;
  if (opts) P.status = opts->status_out;
  cudaError_t e = tk::launch_w(P, w, w_rows, (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

tk_status tk_fwd_w(const float* theta, const float* w, int64_t rows, int64_t n, int64_t w_rows, double p,
                   double lambda, float* out, const tk_opts* opts, tk_stream stream) {
  return run_w(theta, w, nullptr, rows, n, w_rows, p, lambda, out, nullptr, opts, stream, tk::W_FWD);
}

tk_status tk_vjp_w(const float* theta, const float* w, const float* grad_out, int64_t rows, int64_t n,
                   int64_t w_rows, double p, double lambda, float* grad_theta, float* grad_w, const tk_opts* opts,
                   tk_stream stream) {
  return run_w(theta, w, grad_out, rows, n, w_rows, p, lambda, grad_theta, grad_w, opts, stream, tk::W_VJP);
}

tk_status tk_argsort(const float* theta, int64_t rows, int64_t n, int mode, int32_t* perm_out,
                     float* sorted_out, const tk_opts* opts, tk_stream stream) {
  if (rows < 0 || n < 1 || mode < TK_MASK || mode > TK_TOPKMAG) return TK_ERR_INVALID_ARG;
  if (rows == 0) return TK_OK;
  if (theta == nullptr || perm_out == nullptr) return TK_ERR_INVALID_ARG;
  if (n > 0x7fffffff || rows > 0x7fffffffLL) return TK_ERR_UNSUPPORTED;
  tk::Problem P;
  fill(P, theta, rows, n, 1, 0, 0.0, 1.0, mode);
  P.what = tk::W_ARGSORT;
  P.perm_out = perm_out;
  P.sorted_out = sorted_out;
  if (opts) P.status = opts->status_out;
  P.vec4 = (n % 4 == 0) && aligned16(theta);
  if (n > tk::kMaxOnChipN) {
    tk_status s = check_workspace(opts, rows, n);
    if (s != TK_OK) return s;
    cudaError_t el = tk::launch_long(P, opts->workspace, nullptr, true, (cudaStream_t)stream);
    return el == cudaSuccess ? TK_OK : TK_ERR_CUDA;
  }
  cudaError_t e = tk::launch_on_chip(P, (cudaStream_t)stream);
  return e == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

}  // extern "C"
