"""ctypes front end of the CPU oracle (oracle/tko.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
CPU-baseline leg of the benchmark.  The CUDA library never imports this module
and this module never imports the CUDA library.

The shared object is compiled with g++ on first use (or by build()).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tko.cpp")
_LIB = os.path.join(_HERE, "libtko.so")
_lock = threading.Lock()
_lib: Optional[ctypes.CDLL] = None

MASK, TOPK, TOPKMAG = 0, 1, 2
FLAG_RESUM = 1          # solve every pooling sub-problem member by member
FLAG_SINGLE_THREAD = 2  # no OpenMP over rows


def build(force: bool = False) -> str:
    """Compile oracle/tko.cpp into oracle/libtko.so (no-op when up to date)."""
    with _lock:
        if (not force and os.path.exists(_LIB)
                and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
            return _LIB
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
        return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    f32p = ctypes.POINTER(ctypes.c_float)
    f64p = ctypes.POINTER(ctypes.c_double)
    i32p = ctypes.POINTER(ctypes.c_int32)
    i64 = ctypes.c_int64
    lib.tko_num_threads.restype = ctypes.c_int
    lib.tko_argsort.argtypes = [f32p, i64, i64, ctypes.c_int, i32p, f64p]
    lib.tko_fwd.argtypes = [f32p, i64, i64, i64, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                            ctypes.c_int, f64p, i32p, f64p, i32p, i32p]
    lib.tko_vjp.argtypes = [f32p, f32p, i64, i64, i64, ctypes.c_double, ctypes.c_double,
                            ctypes.c_int, ctypes.c_int, f64p]
    lib.tko_dykstra.argtypes = [f32p, i64, i64, i64, ctypes.c_double, ctypes.c_double,
                                ctypes.c_int, ctypes.c_int, ctypes.c_int, f64p, f64p]
    lib.tko_fwd_w.argtypes = [f32p, f64p, i64, i64, i64, ctypes.c_double, ctypes.c_double, f64p, i32p, f64p, i32p, i32p]
    lib.tko_vjp_w.argtypes = [f32p, f64p, f32p, i64, i64, i64, ctypes.c_double, ctypes.c_double, f64p, f64p]
    for fn in (lib.tko_argsort, lib.tko_fwd, lib.tko_vjp, lib.tko_dykstra, lib.tko_fwd_w, lib.tko_vjp_w):
        fn.restype = ctypes.c_int
    _lib = lib
    return lib


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    if a.ndim == 1:
        a = a[None, :]
    if a.ndim != 2:
        raise ValueError("theta must be (rows, n) or (n,)")
    return a


def _ptr(a: Optional[np.ndarray], ty):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ty))
    return a.ctypes.data_as(ctypes.POINTER(ty))


def num_threads() -> int:
    return int(_load().tko_num_threads())


def argsort(theta, mode: int = MASK) -> Tuple[np.ndarray, np.ndarray]:
    """(perm int32, sorted keys float64), both (rows, n)."""
    x = _f32(theta)
    rows, n = x.shape
    perm = np.empty((rows, n), np.int32)
    s = np.empty((rows, n), np.float64)
    rc = _load().tko_argsort(_ptr(x, ctypes.c_float), rows, n, mode, _ptr(perm, ctypes.c_int32),
                             _ptr(s, ctypes.c_double))
    if rc:
        raise ValueError("tko_argsort: invalid argument")
    return perm, s


def fwd(theta, k: int, p: float, lam: float, mode: int = MASK, flags: int = 0,
        details: bool = False):
    """Operator output (rows, n) float64.  details=True also returns a dict with
    perm, v (isotonic solution, sorted coordinates), block_lo, block_hi."""
    x = _f32(theta)
    rows, n = x.shape
    out = np.empty((rows, n), np.float64)
    perm = v = blo = bhi = None
    if details:
        perm = np.empty((rows, n), np.int32)
        v = np.empty((rows, n), np.float64)
        blo = np.empty((rows, n), np.int32)
        bhi = np.empty((rows, n), np.int32)
    rc = _load().tko_fwd(_ptr(x, ctypes.c_float), rows, n, k, p, lam, mode, flags,
                         _ptr(out, ctypes.c_double), _ptr(perm, ctypes.c_int32),
                         _ptr(v, ctypes.c_double), _ptr(blo, ctypes.c_int32),
                         _ptr(bhi, ctypes.c_int32))
    if rc:
        raise ValueError("tko_fwd: invalid argument")
    if details:
        return out, {"perm": perm, "v": v, "block_lo": blo, "block_hi": bhi}
    return out


def vjp(theta, gout, k: int, p: float, lam: float, mode: int = MASK, flags: int = 0) -> np.ndarray:
    x = _f32(theta)
    g = _f32(gout)
    if g.shape != x.shape:
        raise ValueError("cotangent shape differs from theta")
    rows, n = x.shape
    grad = np.empty((rows, n), np.float64)
    rc = _load().tko_vjp(_ptr(x, ctypes.c_float), _ptr(g, ctypes.c_float), rows, n, k, p, lam,
                         mode, flags, _ptr(grad, ctypes.c_double))
    if rc:
        raise ValueError("tko_vjp: invalid argument")
    return grad


def jvp(theta, tangent, k: int, p: float, lam: float, mode: int = MASK) -> np.ndarray:
    """J(theta) tangent per row, assembled from the Jacobian's rows: row i of J is vjp(e_i)
    (Prop. 7 gives the Jacobian; nothing is transposed by hand).  n calls of vjp: small cases."""
    x = _f32(theta)
    v = np.asarray(tangent, np.float64)
    if v.shape != x.shape:
        raise ValueError("tangent shape differs from theta")
    rows, n = x.shape
    out = np.empty((rows, n), np.float64)
    e = np.zeros((rows, n), np.float32)
    for i in range(n):
        e[:, i] = 1.0
        out[:, i] = np.sum(vjp(x, e, k, p, lam, mode) * v, axis=1)
        e[:, i] = 0.0
    return out


def dykstra(theta, k: int, p: float, lam: float, mode: int = MASK, sweeps: int = 100,
            flags: int = 0, return_v: bool = False):
    x = _f32(theta)
    rows, n = x.shape
    out = np.empty((rows, n), np.float64)
    v = np.empty((rows, n), np.float64) if return_v else None
    rc = _load().tko_dykstra(_ptr(x, ctypes.c_float), rows, n, k, p, lam, mode, sweeps, flags,
                             _ptr(out, ctypes.c_double), _ptr(v, ctypes.c_double))
    if rc:
        raise ValueError("tko_dykstra: invalid argument")
    return (out, v) if return_v else out


def _w64(w, rows: int, n: int) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
    if a.ndim == 1:
        a = a[None, :]
    if a.shape not in ((1, n), (rows, n)):
        raise ValueError("w must be (n,), (1, n) or (rows, n)")
    return a


def fwd_w(theta, w, p: float, lam: float, details: bool = False):
    """Relaxed linear maximisation over the permutahedron P(w) (Sec. 3 LP forms, Sec. 4 with
    phi(x) = x): y_R(theta, w), w non-increasing (one vector for all rows, or one per row).
    (rows, n) float64; details=True also returns perm, v, block_lo, block_hi."""
    x = _f32(theta)
    rows, n = x.shape
    ww = _w64(w, rows, n)
    out = np.empty((rows, n), np.float64)
    perm = v = blo = bhi = None
    if details:
        perm = np.empty((rows, n), np.int32); v = np.empty((rows, n), np.float64)
        blo = np.empty((rows, n), np.int32); bhi = np.empty((rows, n), np.int32)
    rc = _load().tko_fwd_w(_ptr(x, ctypes.c_float), _ptr(ww, ctypes.c_double), rows, n, ww.shape[0], p, lam,
                           _ptr(out, ctypes.c_double), _ptr(perm, ctypes.c_int32), _ptr(v, ctypes.c_double),
                           _ptr(blo, ctypes.c_int32), _ptr(bhi, ctypes.c_int32))
    if rc:
        raise ValueError("tko_fwd_w: invalid argument (w must be sorted in non-increasing order)")
    if details:
        return out, {"perm": perm, "v": v, "block_lo": blo, "block_hi": bhi}
    return out


def vjp_w(theta, w, gout, p: float, lam: float, with_w: bool = False):
    """J^T g of y_R(., w) at theta.  with_w=True also returns the cotangent pulled back to w, (rows, n) in
    w's own order (one row per row of theta, also when w is shared)."""
    x = _f32(theta)
    g = _f32(gout)
    rows, n = x.shape
    ww = _w64(w, rows, n)
    grad = np.empty((rows, n), np.float64)
    gw = np.empty((rows, n), np.float64) if with_w else None
    rc = _load().tko_vjp_w(_ptr(x, ctypes.c_float), _ptr(ww, ctypes.c_double), _ptr(g, ctypes.c_float), rows, n,
                           ww.shape[0], p, lam, _ptr(grad, ctypes.c_double),
                           _ptr(gw, ctypes.c_double) if with_w else None)
    if rc:
        raise ValueError("tko_vjp_w: invalid argument")
    return (grad, gw) if with_w else grad


def soft_rank(theta, p: float, lam: float) -> np.ndarray:
    """Relaxed rank (Sec. 3: rank(x) = y(-x, rho), rho = (n, .., 1); rank 1 = largest value)."""
    x = _f32(theta)
    n = x.shape[1]
    return fwd_w(-x, np.arange(n, 0, -1, dtype=np.float64), p, lam)


def soft_sort(theta, p: float, lam: float) -> np.ndarray:
    """Relaxed descending sort (Sec. 3: sort(x) = y(rho, x) = argmax over P(x) of <rho, y>)."""
    x = _f32(theta)
    rows, n = x.shape
    w = -np.sort(-x.astype(np.float64), axis=1)
    rho_v = np.tile(np.arange(n, 0, -1, dtype=np.float32), (rows, 1))
    return fwd_w(rho_v, w, p, lam)


def topk_loss(theta, target, k: int, p: float, lam: float):
    """Smooth top-k loss (Sec. 6, "Smooth top-k loss"): per row
        loss = f(x, 1_k) - <x, t>,   f(x, 1_k) = max_{y in P(1_k)} <y, x> - R(y)
    (Prop. "Relaxed operator" with phi(x) = x, for which the conjugate of f_phi is the indicator of
    the permutahedron P(1_k)), t the one-hot vector of target (t = 0 where target is outside
    [0, n)), R(y) = (lambda/p) sum |y_i|^p.  The maximiser is the relaxed top-k mask y*, so f is
    evaluated at it; the gradient in x is y* - t (same proposition: grad_1 f = y*).
    Returns (loss (rows,), grad (rows, n)), float64."""
    x = _f32(theta)
    rows, n = x.shape
    tgt = np.asarray(target, np.int64).reshape(rows)
    y = fwd(x, k, p, lam, MASK)
    x64 = x.astype(np.float64)
    f = np.sum(y * x64, axis=1) - (lam / p) * np.sum(np.abs(y) ** p, axis=1)
    loss = f.copy()
    grad = y.copy()
    for r in range(rows):
        if 0 <= tgt[r] < n:
            loss[r] -= x64[r, tgt[r]]
            grad[r, tgt[r]] -= 1.0
    return loss, grad


def hard(theta, k: int, mode: int = MASK) -> np.ndarray:
    """The hard operators of Sec. 3 ("Review of operators"): with sigma the (stable, descending)
    argsort of x -- of |x| for topkmag -- topkmask(x) has ones at sigma_1..sigma_k and zeros
    elsewhere, topk(x) = x * topkmask(x), topkmag(x) = x * topkmask(|x|).  This is what the
    "straight-through" use of Sec. 6 runs in the forward pass.  (rows, n) float64."""
    x = _f32(theta)
    rows, n = x.shape
    if not 1 <= k <= n:
        raise ValueError("k out of range")
    perm, _ = argsort(x, mode)
    keep = np.zeros((rows, n), np.float64)
    for r in range(rows):
        keep[r, perm[r, :k]] = 1.0
    return keep if mode == MASK else keep * x.astype(np.float64)
