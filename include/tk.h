/* tk.h -- C ABI of the sm_100a library for p-norm-regularised (smoothed) top-k
 * operators: the batched forward pass and vector-Jacobian product of
 *   topkmask_R, topk_R, topkmag_R   with   R(y) = (lambda/p) * sum_i |y_i|^p,
 * p = 2 or p = 4/3 (any other 1 < p < 2 with the limits below), w = 1_k (k ones
 * followed by zeros); tk_fwd_w / tk_vjp_w take any sorted w.
 *
 * With w = 1_k the isotonic problem the operator reduces to (Prop. 5, Prop. 6) has
 * at most one pooled block, whose value is the root of a non-increasing threshold
 * function of one variable (the capped-simplex condition sum y = k of Sec. 3).
 * By default that root is found per row without sorting, by Newton's iteration
 * on the pieces of the function, and the result is placed by value; when the
 * permutation is asked for (or tk_opts.solver says so) the row is sorted and
 * solved by pool-adjacent-violators on the one block, or by the alternating
 * projections of Algorithm 1.  All three reach the same solution.
 * Paper references are to "Fast, Differentiable and Sparse Top-k: a Convex
 * Analysis Perspective": Sec. 3 = Background, Sec. 4 = Proposed generalized
 * framework, Sec. 5 = Algorithms, App. A = proofs.
 *
 * Conventions shared by every entry point
 *  - All data pointers are DEVICE pointers owned by the caller; row r of a
 *    [rows, n] tensor occupies elements [r*n, r*n + n) (row-major, contiguous).
 *    fp32 values, int32 permutations.
 *  - The library never allocates, frees or synchronises; all work is enqueued
 *    on `stream`.  Scratch memory, when a configuration needs it, is passed in
 *    tk_opts.workspace (size from tk_workspace_bytes).
 *  - Arguments are checked on the host before any launch.  The return value is
 *    a tk_status; nothing throws, exits or traps.  rows == 0 returns TK_OK
 *    without a launch.
 *  - 1 <= k <= n, lambda > 0, p > 1.  q = p/(p-1) within 1e-6 of 2 or 4 (p = 2,
 *    p = 4/3: closed-form block solves, App. A.6) runs on every path.  Any other
 *    p with 2 < q <= 64 (Sec. 7, "sensitivity to the choice of p") runs in all
 *    three modes on rows of up to 16384 elements, with TK_SOLVER_AUTO or
 *    TK_SOLVER_THRESHOLD (no permutation output) or TK_SOLVER_DYKSTRA (the dual
 *    coordinate ascent of App. A.8, every pair solved by a bracketed Newton
 *    iteration; forward pass only).  With the first two solvers rows of up to 128
 *    elements (TK_MASK, TK_TOPK) are sorted and solved by a Newton iteration per
 *    row (forward pass and tk_vjp with or without saved state); longer rows and
 *    TK_TOPKMAG go through the block-per-row threshold solver, and tk_vjp without
 *    saved row state runs that forward pass again, keeping its row state in the
 *    workspace (tk_workspace_bytes; TK_ERR_WORKSPACE without one).  For 1.5 < p < 2 (2 < q < 3) only the forward
 *    pass runs: rho'' is unbounded at 0 and fp32 keys cannot carry the VJP to
 *    1e-5, so tk_vjp / tk_jvp return TK_ERR_UNSUPPORTED.  p > 2 (rho' unbounded
 *    at 0) and q > 64: TK_ERR_UNSUPPORTED.  Outputs must not alias inputs.
 *  - Inputs must be finite.  A NaN/Inf sets TK_FLAG_NONFINITE in *status_out
 *    (when given); that row's output is unspecified, the call still completes.
 */
#ifndef TK_H_
#define TK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque stream handle: a cudaStream_t passed as a pointer (NULL = default stream). */
typedef void *tk_stream;

typedef enum {
  TK_MASK = 0,    /* phi(x) = x:      relaxed top-k mask (Sec. 4, "a relaxed top-k mask")   */
  TK_TOPK = 1,    /* theta * mask_R(theta): relaxed top-k values of a signed input; the hard
                     operator of Sec. 3 with the relaxed mask substituted                   */
  TK_TOPKMAG = 2  /* phi(x) = x^2/2:  relaxed top-k in magnitude (Sec. 4, topkmag_R)        */
} tk_mode;

typedef enum {
  TK_SOLVER_AUTO = 0,     /* the fastest exact path for the request: the threshold form when
                             only values are asked for (rows of more than 8 elements -- 16 for p = 4/3 --, up to
                             32768; longer rows when there are at most 16 of them), else the
                             sort and TK_SOLVER_PAV                                          */
  TK_SOLVER_PAV = 1,      /* sort, then exact pooling of adjacent violators (Sec. 5, App. B.2) */
  TK_SOLVER_DYKSTRA = 2,  /* alternating projections on odd/even pairs (Algorithm 1; for
                             p != 2 the dual block coordinate ascent of App. A.8: closed-form
                             pair step for p = 4/3 with phi(x) = x, a root solve per pair
                             otherwise); rows of up to 131072 elements, those above 16384 with
                             a workspace and p = 2, or p = 4/3 without TK_TOPKMAG, only       */
  TK_SOLVER_THRESHOLD = 3 /* the same exact result as TK_SOLVER_PAV without sorting: root of
                             the capped-simplex threshold function (Sec. 3, P(1_k)); rows of
                             up to 32768 elements (any length when rows <= 16, with a
                             workspace); no permutation output                               */
} tk_solver;

typedef enum {
  TK_OK = 0,
  TK_ERR_INVALID_ARG = 1,   /* null pointer, k out of range, lambda <= 0, p <= 1, ...        */
  TK_ERR_UNSUPPORTED = 2,   /* valid request this build has no kernel for                    */
  TK_ERR_WORKSPACE = 3,     /* workspace missing or smaller than tk_workspace_bytes          */
  TK_ERR_CUDA = 4           /* a CUDA runtime call (launch, attribute) failed                */
} tk_status;

/* bits OR-ed into *tk_opts.status_out by the kernels.  An iteration that stops at its cap is
 * reported here and nowhere else: the host never waits for the device, so no entry point can
 * return it as a status.                                                                       */
#define TK_FLAG_NONFINITE 1      /* some input was NaN or Inf                                */
#define TK_FLAG_NOT_CONVERGED 2  /* an iterative solve stopped at its iteration cap          */
#define TK_FLAG_BOUNDS 4         /* range-checked build of the library only (libtk_bounds.so):
                                    an index left its array; that access was skipped         */

/* What the forward pass found for one row, enough to run the VJP without
 * solving again.  With s the keys in descending order, ranks [a, b) form the
 * single pooled block of the isotonic solution (w = 1_k admits at most one),
 * whose common value is gamma = pivot + offset.  pivot is a value near gamma
 * (the k-th largest key on the sorted paths, the last pivot of the iteration on
 * the threshold path), kept apart from offset so that key - gamma can be formed
 * as (key - pivot) - offset without cancellation; every consumer classifies a
 * key by that expression: capped at width or more, pooled above 0, zero else.
 * a == b == k means no pooled block: every key >= pivot is a top singleton,
 * every other key a bottom singleton (offset is 0 then).                       */
typedef struct {
  float pivot;
  float offset;
  int32_t a;
  int32_t b;
} tk_rowstate;

typedef struct {
  int solver;              /* tk_solver                                                       */
  int sweeps;              /* Dykstra sweeps; <= 0 means 100 (the count used in Sec. 5)       */
  int32_t *perm_out;       /* [rows*n] sorted rank -> original index, or NULL                 */
  tk_rowstate *state_out;  /* tk_fwd_ex: [rows] written.  tk_vjp: [rows] read (saved by a
                              forward call with identical arguments), or NULL = recompute    */
  void *workspace;         /* device scratch, 256-byte aligned, or NULL                       */
  size_t workspace_bytes;
  int32_t *status_out;     /* one device word, OR of TK_FLAG_*; the caller zeroes it          */
  int flags;               /* OR of TK_OPT_*                                                  */
  float tol;               /* TK_SOLVER_DYKSTRA only.  0: exactly `sweeps` sweeps (Sec. 5 uses fixed
                              counts).  > 0: the sweeps of a row end as soon as no entry of its
                              iterate (p = 2) / none of its duals (p = 4/3) moved by more than tol
                              in any projection of a sweep; `sweeps` is then the cap, and a row that
                              reaches it sets TK_FLAG_NOT_CONVERGED (a tol below the fp32 spacing of the keys
                              is never met).  Rows of up to 16384 elements
                              (longer: TK_ERR_UNSUPPORTED); negative or non-finite: invalid       */
} tk_opts;

/* tk_fwd_ex only: the "straight-through" use of Sec. 6 (experiments, weight pruning).  out
 * receives the HARD operator of Sec. 3 -- topkmask: ones at the k largest entries; topk: theta
 * there, zero elsewhere; topkmag: the same on |theta| -- equal keys kept in ascending index,
 * while state_out still receives the row state of the RELAXED operator, so that tk_vjp / tk_jvp
 * from that state give the relaxed operator's derivative for the backward pass.  The hard
 * output is read off the permutation: perm_out is required (TK_ERR_INVALID_ARG without it), and
 * the solver must be one that sorts (not TK_SOLVER_THRESHOLD; general p has no permutation
 * output: TK_ERR_UNSUPPORTED).                                                              */
#define TK_OPT_STRAIGHT_THROUGH 1

/* Scratch bytes tk_fwd_ex / tk_vjp / tk_argsort need for this shape: 0 for rows
 * of up to 16384 elements.  Rows of 16385..32768 elements need it only when a
 * permutation is returned (perm_out, tk_argsort), tk_vjp has no saved row
 * state, or the solver is TK_SOLVER_DYKSTRA; the plain forward pass and the VJP
 * from state run without.  A general p needs rows * sizeof(tk_rowstate) bytes for
 * tk_vjp without saved state (rows above 128 elements, or TK_TOPKMAG).  Longer rows always need it (the threshold path for
 * at most 16 such rows keeps its per-block partial sums there; the sorting
 * pipeline its buffers).  solver as in tk_opts.                                */
size_t tk_workspace_bytes(int64_t rows, int64_t n, int64_t k, double p, int mode, int solver);

/* Forward pass (Prop. 2 with Prop. 5 / Prop. 6): out[r, :] = operator(theta[r, :]).
 * theta, out: device, [rows*n] fp32.  Fails with TK_ERR_WORKSPACE for shapes that
 * need scratch (use tk_fwd_ex).                                                 */
tk_status tk_fwd(const float *theta, int64_t rows, int64_t n, int64_t k, double p, double lambda,
                 int mode, float *out, tk_stream stream);

/* Forward pass with options (solver choice, permutation / row state outputs,
 * workspace, status word).  opts may be NULL (= tk_fwd).                        */
tk_status tk_fwd_ex(const float *theta, int64_t rows, int64_t n, int64_t k, double p,
                    double lambda, int mode, float *out, const tk_opts *opts, tk_stream stream);

/* Vector-Jacobian product (Prop. 7 chained through y = grad R*(x - u)):
 * grad_theta[r, :] = J(theta[r, :])^T grad_out[r, :].  All device, [rows*n] fp32.
 * With opts->state_out from a forward call nothing is solved again.  Without it the
 * row is solved again: by the sort-free forward pass when opts->workspace has room
 * for the row state (rows * sizeof(tk_rowstate) bytes, 256-byte aligned; rows of up
 * to 32768 elements), inside a sorting kernel otherwise.                         */
tk_status tk_vjp(const float *theta, const float *grad_out, int64_t rows, int64_t n, int64_t k,
                 double p, double lambda, int mode, float *grad_theta, const tk_opts *opts,
                 tk_stream stream);

/* Jacobian-vector product (the Jacobian of Prop. 7 chained through y = grad R*(x - u),
 * applied to a tangent instead of a cotangent): out_tangent[r, :] = J(theta[r, :]) tangent[r, :].
 * All device, [rows*n] fp32.  opts->state_out must hold the row state a forward call saved
 * (TK_ERR_UNSUPPORTED without it); rows of more than 32768 elements also need opts->workspace.
 * For TK_MASK and TK_TOPKMAG the Jacobian is symmetric and the result equals tk_vjp's.        */
tk_status tk_jvp(const float *theta, const float *tangent, int64_t rows, int64_t n, int64_t k,
                 double p, double lambda, int mode, float *out_tangent, const tk_opts *opts,
                 tk_stream stream);

/* Smooth top-k loss (Sec. 6, "Smooth top-k loss"; a Fenchel-Young loss built on Prop. "Relaxed
 * operator" with phi(x) = x):
 *   loss[r] = f(theta_r, 1_k) - theta[r, target[r]],
 *   f(x, 1_k) = max_{y in P(1_k)} <y, x> - R(y) = <y*, x> - (lambda/p) sum_i (y*_i)^p,
 * y* the relaxed top-k mask of the row, and its gradient in theta (grad_1 f = y*):
 *   grad[r, :] = y* - onehot(target[r]).
 * theta: device [rows*n] fp32; target: device [rows] int32 class index, a value outside [0, n)
 * (or target == NULL) means no target for that row: loss = f, grad = y*; loss: device [rows]
 * fp32; grad: device [rows*n] fp32 (it also serves as the buffer the mask is computed in).
 * opts as for tk_fwd_ex (solver, workspace, status word, row state of the mask); every limit of
 * tk_fwd_ex in TK_MASK mode applies.  Two launches: the forward pass, then one pass over
 * (theta, y*) that reduces each row and subtracts the target.                                  */
tk_status tk_topk_loss(const float *theta, const int32_t *target, int64_t rows, int64_t n, int64_t k,
                       double p, double lambda, float *loss, float *grad, const tk_opts *opts,
                       tk_stream stream);

/* The operator along the slow axis of a matrix (Sec. 6, sparse MoE with expert-choice routing:
 * every expert takes its top-k over the tokens, from a [tokens, experts] score matrix).
 * theta, out (and grad_out, grad_theta): device, n rows of `cols` fp32 values, row i starting at
 * element i * ld (ld >= cols, the same for every array of a call); problem c is column c:
 *   out[:, c] = operator(theta[:, c]),   grad_theta[:, c] = J(theta[:, c])^T grad_out[:, c].
 * The columns are transposed into opts->workspace (tk_cols_workspace_bytes, 256-byte aligned;
 * TK_ERR_WORKSPACE without it), the row kernels run there, and the result is transposed back:
 * one extra read and write of every array.  n <= 16384; cols <= 2^21; opts otherwise as for
 * tk_fwd_ex / tk_vjp with rows = cols (state_out: one record per column; perm_out: [cols*n],
 * contiguous per column).  tk_vjp_cols reads the workspace copy of theta that tk_fwd_cols left
 * there when opts->state_out is given and theta == NULL is passed; with theta given it is
 * transposed again.                                                                          */
size_t tk_cols_workspace_bytes(int64_t n, int64_t cols);
tk_status tk_fwd_cols(const float *theta, int64_t n, int64_t cols, int64_t ld, int64_t k, double p,
                      double lambda, int mode, float *out, const tk_opts *opts, tk_stream stream);
tk_status tk_vjp_cols(const float *theta, const float *grad_out, int64_t n, int64_t cols, int64_t ld,
                      int64_t k, double p, double lambda, int mode, float *grad_theta,
                      const tk_opts *opts, tk_stream stream);

/* Relaxed linear maximisation over the permutahedron P(w) of any sorted vector w (Sec. 3, LP forms
 * of sort and rank; Sec. 4, the relaxed operator with phi(x) = x; Prop. 5 for its reduction to
 * isotonic optimisation, solved here by pool-adjacent-violators with many blocks, App. B.2):
 *   out[r, :] = argmax_{y in P(w_r)} <theta[r, :], y> - R(y).
 * w_r = (1,..,1,0,..,0) gives the relaxed top-k mask of tk_fwd; w = (n, n-1, .., 1) applied to
 * -x gives the relaxed rank of x (rank 1 = largest value); theta = (n, .., 1) with w_r = x_r
 * sorted gives the relaxed descending sort of x_r.
 * theta, out: device [rows*n] fp32.  w: device fp32, [n] shared by every row (w_rows = 1) or
 * [rows*n] (w_rows = rows); every row of w must be in non-increasing order (it is not checked:
 * an unsorted w gives an unspecified result).  p = 2 or p = 4/3, n <= 2048 (else
 * TK_ERR_UNSUPPORTED).  opts may carry status_out; the other fields must be unset.
 * tk_vjp_w: grad_theta[r, :] = J(theta[r, :])^T grad_out[r, :], the Jacobian of Prop. 7 (block
 * diagonal over the pooled blocks) in theta; the row is sorted and solved again.  grad_w (may be
 * NULL): device [rows*n], the cotangent pulled back to w, per row and in w's own order -- inside a
 * pooled block B the value solves sum_B rho(s_i - gamma) = sum_B w_i, so every w_j of the block
 * receives sum_B rho' g / sum_B rho'.  It is what the relaxed sort needs, whose input enters as w;
 * for a w shared by all rows the caller adds the rows up.                                         */
tk_status tk_fwd_w(const float *theta, const float *w, int64_t rows, int64_t n, int64_t w_rows, double p,
                   double lambda, float *out, const tk_opts *opts, tk_stream stream);
tk_status tk_vjp_w(const float *theta, const float *w, const float *grad_out, int64_t rows, int64_t n,
                   int64_t w_rows, double p, double lambda, float *grad_theta, float *grad_w,
                   const tk_opts *opts, tk_stream stream);

/* Segmented stable descending argsort (Sec. 3, argsort/sort): per row,
 * perm_out[i] = index of the i-th largest key (theta, or |theta| for
 * TK_TOPKMAG), equal keys in ascending index, -0 == +0.  sorted_out (may be
 * NULL) receives the keys in that order.  opts may carry a workspace.           */
tk_status tk_argsort(const float *theta, int64_t rows, int64_t n, int mode, int32_t *perm_out,
                     float *sorted_out, const tk_opts *opts, tk_stream stream);

/* Forward pass that brings its own scratch memory.  The paper has no counterpart
 * to this entry point; it exists for callers that cannot allocate device memory
 * when they need the operator: a plugin inside an application that owns the
 * allocator, a real-time loop that must not hit cudaMalloc's implicit device
 * synchronisation, a process whose memory pool is fully committed.  Such callers
 * can use tk_fwd for rows of up to 32768 elements (which needs no scratch), but
 * tk_fwd_ex wants a workspace for longer rows; this call does not.
 *
 * Arguments, layout and results are those of tk_fwd (all pointers device
 * pointers owned by the caller; out[r, :] = operator(theta[r, :]); work is
 * enqueued on `stream`).  Rows of up to 32768 elements are passed straight to
 * tk_fwd.  Longer rows run the global-memory pipeline of tk_fwd_ex on a scratch
 * array compiled into the library: TK_NOALLOC_SCRATCH_BYTES of device memory
 * that a GPU holds from the moment the CUDA runtime loads the library's module
 * on it until the process exits.  The call never asks an allocator for memory
 * (no cudaMalloc, cudaFree or allocating library routine).
 *
 *  - Limit: rows * n <= TK_NOALLOC_MAX_ELEMENTS (and the scratch the shape needs
 *    must fit the array); anything larger returns TK_ERR_WORKSPACE before any
 *    launch.  Use tk_fwd_ex with your own workspace for bigger problems.
 *  - The first call on a device looks up the array's device address
 *    (cudaGetSymbolAddress) with that device current.  With CUDA's default lazy
 *    module loading that lookup is also what loads the module, and with it
 *    reserves the array, on that device: it is the one call that can fail with
 *    TK_ERR_CUDA when the device has no room left.  Make it once at start-up,
 *    before the memory pool is committed and outside of any stream capture.
 *    The address is not looked up again: after cudaDeviceReset it is stale and
 *    this entry point must not be used in that process any more.
 *  - All calls on a device share the one array.  It keeps whatever the previous
 *    call left in it, which is harmless (every word is written before it is read
 *    within a call), but two calls whose kernels overlap on the GPU -- different
 *    streams, or concurrent host threads -- race on it and produce garbage.
 *    Serialise them on one stream.                                              */
#define TK_NOALLOC_MAX_ELEMENTS (1 << 18)
#define TK_NOALLOC_SCRATCH_BYTES (8u << 20)
tk_status tk_fwd_noalloc(const float *theta, int64_t rows, int64_t n, int64_t k, double p,
                         double lambda, int mode, float *out, tk_stream stream);

const char *tk_status_string(int status);

/* Library build tag, e.g. "tk 0.1 sm_100a".                                     */
const char *tk_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TK_H_ */
