"""Thin ctypes binding of libtk.so: argument marshalling only.

Every function here has the name and the arguments of its C counterpart in
include/tk.h; tensors are torch CUDA tensors used purely as device buffers and
work is enqueued on torch's current stream.  There is no CPU path: loading
fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtk.so")

TK_MASK, TK_TOPK, TK_TOPKMAG = 0, 1, 2
TK_SOLVER_AUTO, TK_SOLVER_PAV, TK_SOLVER_DYKSTRA, TK_SOLVER_THRESHOLD = 0, 1, 2, 3
TK_OK = 0
TK_ERR_INVALID_ARG, TK_ERR_UNSUPPORTED, TK_ERR_WORKSPACE, TK_ERR_CUDA = 1, 2, 3, 4
TK_FLAG_NONFINITE, TK_FLAG_NOT_CONVERGED, TK_FLAG_BOUNDS = 1, 2, 4
TK_OPT_STRAIGHT_THROUGH = 1
ROWSTATE_BYTES = 16

EXPORTS = ("tk_version", "tk_status_string", "tk_workspace_bytes", "tk_fwd", "tk_fwd_ex", "tk_vjp",
           "tk_jvp", "tk_argsort", "tk_fwd_noalloc", "tk_topk_loss",
           "tk_cols_workspace_bytes", "tk_fwd_cols", "tk_vjp_cols", "tk_fwd_w", "tk_vjp_w")
TK_NOALLOC_MAX_ELEMENTS = 1 << 18


class TkOpts(ctypes.Structure):
    _fields_ = [
        ("solver", ctypes.c_int),
        ("sweeps", ctypes.c_int),
        ("perm_out", ctypes.c_void_p),
        ("state_out", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
        ("status_out", ctypes.c_void_p),
        ("flags", ctypes.c_int),
        ("tol", ctypes.c_float),
    ]


class TkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib: Optional[ctypes.CDLL] = None


def use_library(path: str) -> None:
    """Bind the calls below to another build of the library (the range-checked libtk_bounds.so);
    takes effect at the next load()."""
    global _lib, LIB_PATH
    LIB_PATH = path
    _lib = None


def load() -> ctypes.CDLL:
    """Load libtk.so; raises if it is missing (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2302_01425_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
    lib.tk_version.restype = ctypes.c_char_p
    lib.tk_status_string.restype = ctypes.c_char_p
    lib.tk_status_string.argtypes = [ci]
    lib.tk_workspace_bytes.restype = ctypes.c_size_t
    lib.tk_workspace_bytes.argtypes = [i64, i64, i64, dbl, ci, ci]
    lib.tk_fwd.restype = ci
    lib.tk_fwd.argtypes = [vp, i64, i64, i64, dbl, dbl, ci, vp, vp]
    lib.tk_fwd_noalloc.restype = ci
    lib.tk_fwd_noalloc.argtypes = [vp, i64, i64, i64, dbl, dbl, ci, vp, vp]
    lib.tk_fwd_ex.restype = ci
    lib.tk_fwd_ex.argtypes = [vp, i64, i64, i64, dbl, dbl, ci, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_vjp.restype = ci
    lib.tk_vjp.argtypes = [vp, vp, i64, i64, i64, dbl, dbl, ci, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_jvp.restype = ci
    lib.tk_jvp.argtypes = [vp, vp, i64, i64, i64, dbl, dbl, ci, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_topk_loss.restype = ci
    lib.tk_topk_loss.argtypes = [vp, vp, i64, i64, i64, dbl, dbl, vp, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_cols_workspace_bytes.restype = ctypes.c_size_t
    lib.tk_cols_workspace_bytes.argtypes = [i64, i64]
    lib.tk_fwd_cols.restype = ci
    lib.tk_fwd_cols.argtypes = [vp, i64, i64, i64, i64, dbl, dbl, ci, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_vjp_cols.restype = ci
    lib.tk_vjp_cols.argtypes = [vp, vp, i64, i64, i64, i64, dbl, dbl, ci, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_fwd_w.restype = ci
    lib.tk_fwd_w.argtypes = [vp, vp, i64, i64, i64, dbl, dbl, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_vjp_w.restype = ci
    lib.tk_vjp_w.argtypes = [vp, vp, vp, i64, i64, i64, dbl, dbl, vp, vp, ctypes.POINTER(TkOpts), vp]
    lib.tk_argsort.restype = ci
    lib.tk_argsort.argtypes = [vp, i64, i64, ci, vp, vp, ctypes.POINTER(TkOpts), vp]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().tk_status_string(int(status)).decode()


def version() -> str:
    return load().tk_version().decode()


def _dev(t: Optional[torch.Tensor], dtype, what: str, need: int = 0) -> Optional[int]:
    """Device address of a buffer; `need` = the elements the call will touch (the C side takes rows
    and n apart from the buffers, so a short tensor would be read or written out of bounds)."""
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{what}: expected a contiguous CUDA tensor of {dtype}")
    if t.numel() < need:
        raise ValueError(f"{what}: {t.numel()} elements, the call needs {need}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _opts(solver=TK_SOLVER_AUTO, sweeps=0, perm_out=None, state=None, workspace=None,
          status_out=None, flags=0, rows=0, n=0, tol=0.0) -> TkOpts:
    o = TkOpts()
    o.flags = int(flags)
    o.tol = float(tol)
    o.solver, o.sweeps = int(solver), int(sweeps)
    o.perm_out = _dev(perm_out, torch.int32, "perm_out", rows * n)
    o.state_out = None if state is None else _dev(state, torch.uint8, "state", rows * ROWSTATE_BYTES)
    o.workspace = None if workspace is None else _dev(workspace, torch.uint8, "workspace")
    o.workspace_bytes = 0 if workspace is None else workspace.numel()
    o.status_out = _dev(status_out, torch.int32, "status_out", 1)
    return o


def new_state(rows: int, device="cuda") -> torch.Tensor:
    """Device buffer for `rows` tk_rowstate records."""
    return torch.empty(rows * ROWSTATE_BYTES, dtype=torch.uint8, device=device)


def tk_workspace_bytes(rows: int, n: int, k: int, p: float, mode: int, solver: int = 0) -> int:
    return int(load().tk_workspace_bytes(rows, n, k, p, mode, solver))


def tk_fwd(theta: torch.Tensor, rows: int, n: int, k: int, p: float, lam: float, mode: int,
           out: torch.Tensor) -> None:
    rc = load().tk_fwd(_dev(theta, torch.float32, "theta", rows * n), rows, n, k, p, lam, mode,
                       _dev(out, torch.float32, "out", rows * n), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_fwd")


def tk_fwd_noalloc(theta: torch.Tensor, rows: int, n: int, k: int, p: float, lam: float, mode: int,
                   out: torch.Tensor) -> None:
    """tk_fwd for callers that cannot allocate: long rows use the scratch array built into
    the library (rows * n <= TK_NOALLOC_MAX_ELEMENTS; calls must not overlap on the GPU)."""
    rc = load().tk_fwd_noalloc(_dev(theta, torch.float32, "theta", rows * n), rows, n, k, p, lam, mode,
                               _dev(out, torch.float32, "out", rows * n), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_fwd_noalloc")


def tk_fwd_ex(theta, rows, n, k, p, lam, mode, out, *, solver=TK_SOLVER_AUTO, sweeps=0,
              perm_out=None, state_out=None, workspace=None, status_out=None, flags=0, tol=0.0) -> None:
    o = _opts(solver, sweeps, perm_out, state_out, workspace, status_out, flags, rows=rows, n=n, tol=tol)
    rc = load().tk_fwd_ex(_dev(theta, torch.float32, "theta", rows * n), rows, n, k, p, lam, mode,
                          _dev(out, torch.float32, "out", rows * n), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_fwd_ex")


def tk_vjp(theta, grad_out, rows, n, k, p, lam, mode, grad_theta, *, state=None, workspace=None,
           status_out=None) -> None:
    o = _opts(state=state, workspace=workspace, status_out=status_out, rows=rows, n=n)
    rc = load().tk_vjp(_dev(theta, torch.float32, "theta", rows * n), _dev(grad_out, torch.float32, "grad_out", rows * n),
                       rows, n, k, p, lam, mode, _dev(grad_theta, torch.float32, "grad_theta", rows * n),
                       ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_vjp")


def tk_jvp(theta, tangent, rows, n, k, p, lam, mode, out_tangent, *, state, workspace=None,
           status_out=None) -> None:
    o = _opts(state=state, workspace=workspace, status_out=status_out, rows=rows, n=n)
    rc = load().tk_jvp(_dev(theta, torch.float32, "theta", rows * n), _dev(tangent, torch.float32, "tangent", rows * n),
                       rows, n, k, p, lam, mode, _dev(out_tangent, torch.float32, "out_tangent", rows * n),
                       ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_jvp")


def tk_topk_loss(theta, target, rows, n, k, p, lam, loss, grad, *, solver=TK_SOLVER_AUTO, sweeps=0,
                 state_out=None, workspace=None, status_out=None) -> None:
    o = _opts(solver, sweeps, None, state_out, workspace, status_out, rows=rows, n=n)
    rc = load().tk_topk_loss(_dev(theta, torch.float32, "theta", rows * n), _dev(target, torch.int32, "target", rows),
                             rows, n, k, p, lam, _dev(loss, torch.float32, "loss", rows),
                             _dev(grad, torch.float32, "grad", rows * n), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_topk_loss")


def tk_cols_workspace_bytes(n: int, cols: int) -> int:
    return int(load().tk_cols_workspace_bytes(n, cols))


def tk_fwd_cols(theta, n, cols, ld, k, p, lam, mode, out, *, workspace, solver=TK_SOLVER_AUTO, sweeps=0,
                perm_out=None, state_out=None, status_out=None, flags=0) -> None:
    o = _opts(solver, sweeps, perm_out, state_out, workspace, status_out, flags, rows=cols, n=n)
    span = (n - 1) * ld + cols if n > 0 else 0          # last element touched of an [n, cols] matrix with leading dimension ld
    rc = load().tk_fwd_cols(_dev(theta, torch.float32, "theta", span), n, cols, ld, k, p, lam, mode,
                            _dev(out, torch.float32, "out", span), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_fwd_cols")


def tk_vjp_cols(theta, grad_out, n, cols, ld, k, p, lam, mode, grad_theta, *, workspace, state=None,
                status_out=None) -> None:
    o = _opts(state=state, workspace=workspace, status_out=status_out, rows=cols, n=n)
    span = (n - 1) * ld + cols if n > 0 else 0
    rc = load().tk_vjp_cols(_dev(theta, torch.float32, "theta", span), _dev(grad_out, torch.float32, "grad_out", span),
                            n, cols, ld, k, p, lam, mode, _dev(grad_theta, torch.float32, "grad_theta", span),
                            ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_vjp_cols")


def tk_argsort(theta, rows, n, mode, perm_out, sorted_out=None, *, workspace=None,
               status_out=None) -> None:
    o = _opts(workspace=workspace, status_out=status_out)
    rc = load().tk_argsort(_dev(theta, torch.float32, "theta", rows * n), rows, n, mode,
                           _dev(perm_out, torch.int32, "perm_out", rows * n),
                           _dev(sorted_out, torch.float32, "sorted_out", rows * n), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_argsort")


def tk_fwd_w(theta, w, rows, n, p, lam, out, *, status_out=None) -> None:
    """w: [n] (shared by every row) or [rows, n], every row non-increasing."""
    w_rows = 1 if w.numel() == n and rows != 1 else (rows if w.numel() >= rows * n else 1)
    o = _opts(status_out=status_out)
    rc = load().tk_fwd_w(_dev(theta, torch.float32, "theta", rows * n), _dev(w, torch.float32, "w", w_rows * n),
                         rows, n, w_rows, p, lam, _dev(out, torch.float32, "out", rows * n), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_fwd_w")


def tk_vjp_w(theta, w, grad_out, rows, n, p, lam, grad_theta, *, grad_w=None, status_out=None) -> None:
    """grad_w (optional): [rows, n], the cotangent pulled back to w (per row, in w's order)."""
    w_rows = 1 if w.numel() == n and rows != 1 else (rows if w.numel() >= rows * n else 1)
    o = _opts(status_out=status_out)
    rc = load().tk_vjp_w(_dev(theta, torch.float32, "theta", rows * n), _dev(w, torch.float32, "w", w_rows * n),
                         _dev(grad_out, torch.float32, "grad_out", rows * n), rows, n, w_rows, p, lam,
                         _dev(grad_theta, torch.float32, "grad_theta", rows * n),
                         _dev(grad_w, torch.float32, "grad_w", rows * n), ctypes.byref(o), _stream())
    if rc != TK_OK:
        raise TkError(rc, "tk_vjp_w")
